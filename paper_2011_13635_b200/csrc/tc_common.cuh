// Building blocks shared by the tensor-core kernels (sm_100a): PTX wrappers for mbarriers, TMA
// tile copies, tcgen05 MMA / commit / tensor-memory loads, the shared-memory matrix descriptor,
// the per-warp staging buffer that turns one-row-per-lane registers into coalesced row-segment
// stores, and the host-side builder of rank-4 tensor maps.
#pragma once
#include <cuda.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <mutex>
#include <unordered_map>

#include "common.cuh"
#include "../../include/mslt.h"

namespace mslt {
namespace {

constexpr int BM = 128;           // rows of an output tile = TMEM lanes
constexpr int BK = 64;            // k extent of a stage: 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;        // k extent of one tcgen05.mma for 16-bit operands
constexpr int MAX_STAGES = 8;
constexpr int A_STAGE_BYTES = BM * BK * 2;
constexpr int NUM_EPI_WARPS = 8;
constexpr int NUM_THREADS = 64 + 32 * NUM_EPI_WARPS;
constexpr int STAGING_BYTES = 4096;  // per epilogue warp
constexpr uint32_t TMEM_COLS = 512;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000ll;  // about 2 s of SM clock (the default limit)

// ---- PTX wrappers -----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
// SM cycle counter: cheap to read, which matters because every bounded wait samples it
__device__ __forceinline__ long long now_cycles() { return clock64(); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false when the limit ran out or another role already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = now_cycles();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++spins & 255u) == 0u) {
      if (*abort_flag) return false;
      if (now_cycles() - t0 > *reinterpret_cast<volatile long long*>(abort_flag + 1)) {
        *abort_flag = 1;
        atomicOr(status, ST_WAIT_TIMEOUT);
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
// Tile store from shared memory (the tile in the tensor map's swizzled layout) to global memory;
// the part of the box outside the tensor is not written.  c0 * element size must be a multiple of
// 16 bytes and no coordinate negative.  Completion is tracked by the thread's bulk async-groups.
__device__ __forceinline__ void tma_store_4d(const CUtensorMap* map, uint32_t src, int c0, int c1, int c2, int c3) {
  asm volatile("cp.async.bulk.tensor.4d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4, %5}], [%1];"
               ::"l"(map), "r"(src), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
               : "memory");
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the issuing thread's tile stores have all read their shared memory / have all completed
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// makes this thread's shared-memory writes visible to the copy engine
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// ---- CTA-pair (cta_group::2) forms: the two CTAs of a cluster work on one 256-row tile ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// the copy lands in this CTA's shared memory; its bytes are counted on the leader CTA's barrier
__device__ __forceinline__ void tma_load_4d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster,
                                                 int c0, int c1, int c2, int c3) {
  asm volatile(
      "cp.async.bulk.tensor.4d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4, %5, %6}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
      : "memory");
}
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {  // arrives on the barrier in both CTAs
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(bar), "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}

__device__ __forceinline__ void tc_fence_before() {
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_after() {
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
}
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 consecutive accumulator columns of this lane's row, as 16 (even, odd) column pairs
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float2 (&w)[16]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; i++) w[i] = make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
}
__device__ __forceinline__ float2 splat2(float c) { return make_float2(c, c); }

// The same read split in two, so that the next chunk's read is in flight while this chunk is worked
// on: after tc_ld32_issue the registers are not valid until tc_ld32_wait has returned.  The wait
// names the registers as in/out operands so that no use of them can be scheduled above it.
__device__ __forceinline__ void tc_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
        "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
        "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
        "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_ld32_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]),
                 "+r"(r[15])
               :
               : "memory");
  // the second half of the registers is tied to the same point in the instruction stream
  asm volatile(""
               : "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]),
                 "+r"(r[23]), "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]),
                 "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// Shared-memory matrix descriptor for a 128-byte-swizzled tile whose rows are 128 bytes apart and
// whose 8-row groups are 1024 bytes apart.  lbo_bytes: distance between 64-element column blocks
// of an MN-major operand (ignored by the hardware for K-major swizzled tiles).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((1024u >> 4) & 0x3FFFu) << 32;  // stride between 8-row groups
  d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                         // 128-byte swizzle
  return d;
}

__device__ __forceinline__ float2 bf162_to_f2(uint32_t h) {
  return make_float2(__uint_as_float(h << 16), __uint_as_float(h & 0xffff0000u));
}

// Staging buffer of one epilogue warp: 32 rows of 64 bytes (2 KB).  Lane r writes its row as four
// 16-byte pieces; the slot function permutes the pieces so that both this
// row-per-lane write and the row-segment-per-quarter-warp read that follows are free of bank
// conflicts.  Bytes 2048.. of the warp's 4 KB hold the bias values of the warp's columns.
__device__ __forceinline__ uint32_t slot_b16(int r, int c) {  // c in 0..3: pieces of 8 bf16 or 4 floats
  return (uint32_t)(r * 64 + ((c ^ ((r >> 1) & 3)) << 4));
}

// Writes a 32 x 32 chunk (lane = row, v = its 32 columns) to `base` (row-major, leading dimension
// ldd, element (m_warp + row, n0 + col)) with coalesced 16-byte stores.
__device__ __forceinline__ void stage_store_bf16(uint8_t* stg, int lane, const float2 (&w)[16], bf16* base,
                                                 long long ldd, int m_warp, int n0, int M, int N,
                                                 int vec_ok) {
#pragma unroll
  for (int c = 0; c < 4; c++) {
    uint4 pk;
    __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&pk);
#pragma unroll
    for (int e = 0; e < 4; e++) h[e] = __float22bfloat162_rn(w[4 * c + e]);
    *reinterpret_cast<uint4*>(stg + slot_b16(lane, c)) = pk;
  }
  __syncwarp();
#pragma unroll
  for (int it = 0; it < 4; it++) {
    const int row = it * 8 + (lane >> 2), c = lane & 3;
    const uint4 val = *reinterpret_cast<const uint4*>(stg + slot_b16(row, c));
    const int mm = m_warp + row, nn = n0 + c * 8;
    if (mm < M && nn < N) {
      bf16* dst = base + (long long)mm * ldd + nn;
      if (vec_ok && nn + 8 <= N) {
        *reinterpret_cast<uint4*>(dst) = val;
      } else {
        const bf16* e8 = reinterpret_cast<const bf16*>(&val);
#pragma unroll
        for (int e = 0; e < 8; e++)
          if (nn + e < N) dst[e] = e8[e];
      }
    }
  }
  __syncwarp();
}

// fp32 output: the same 2 KB transposer, used twice for 16 columns each.
__device__ __forceinline__ void stage_store_f32(uint8_t* stg, int lane, const float2 (&w)[16], float* base,
                                                long long ldd, int m_warp, int n0, int M, int N, int vec_ok,
                                                int accumulate) {
#pragma unroll
  for (int half = 0; half < 2; half++) {
#pragma unroll
    for (int c = 0; c < 4; c++)
      *reinterpret_cast<float4*>(stg + slot_b16(lane, c)) =
          make_float4(w[8 * half + 2 * c].x, w[8 * half + 2 * c].y, w[8 * half + 2 * c + 1].x,
                      w[8 * half + 2 * c + 1].y);
    __syncwarp();
#pragma unroll
    for (int it = 0; it < 4; it++) {
      const int row = it * 8 + (lane >> 2), c = lane & 3;
      const float4 val = *reinterpret_cast<const float4*>(stg + slot_b16(row, c));
      const int mm = m_warp + row, nn = n0 + half * 16 + c * 4;
      if (mm < M && nn < N) {
        float* dst = base + (long long)mm * ldd + nn;
        if (vec_ok && nn + 4 <= N) {
          if (accumulate)
            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(val.x), "f"(val.y),
                         "f"(val.z), "f"(val.w)
                         : "memory");
          else
            *reinterpret_cast<float4*>(dst) = val;
        } else {
          const float e4[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
          for (int e = 0; e < 4; e++)
            if (nn + e < N) {
              if (accumulate) atomicAdd(dst + e, e4[e]); else dst[e] = e4[e];
            }
        }
      }
    }
    __syncwarp();
  }
}

// Hand-over between the two epilogue warps of a TMEM lane quarter: publish my sequence number
// after my shared-memory writes, then wait (bounded) until the partner has published the same.
__device__ __forceinline__ bool pair_sync(volatile int* flags, int me, int other, int seq, int lane,
                                          volatile int* abort_flag, int* status) {
  __syncwarp();
  int ok = 1;
  if (lane == 0) {
    __threadfence_block();
    flags[me] = seq;
    const long long t0 = now_cycles();
    uint32_t spins = 0;
    while (flags[other] < seq) {
      if ((++spins & 255u) == 0u) {
        if (*abort_flag) { ok = 0; break; }
        if (now_cycles() - t0 > *reinterpret_cast<volatile long long*>(abort_flag + 1)) {
          *abort_flag = 1;
          atomicOr(status, ST_WAIT_TIMEOUT);
          ok = 0;
          break;
        }
      }
    }
    __threadfence_block();
  }
  ok = __shfl_sync(0xffffffffu, ok, 0);
  return ok != 0;
}

// ---- host side: tensor maps and launch ------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  });
  return fn;
}

struct MapKey {
  const void* ptr;
  long long rows, K, rs, ks, bo, bi;
  int hdiv, nb, box_rows;
  bool operator==(const MapKey& o) const { return memcmp(this, &o, sizeof(MapKey)) == 0; }
};
struct MapKeyHash {
  size_t operator()(const MapKey& k) const {
    const uint64_t* w = reinterpret_cast<const uint64_t*>(&k);
    uint64_t h = 1469598103934665603ull;
    for (size_t i = 0; i < sizeof(MapKey) / 8; i++) h = (h ^ w[i]) * 1099511628211ull;
    return (size_t)h;
  }
};
struct MapVal {
  CUtensorMap map;
  int perm[3];
};

// Builds (or fetches) the rank-4 tensor map of one operand: dim 0 is the contiguous index (k for a
// K-major operand, the row index otherwise); the other matrix index and the two batch indices
// follow in order of increasing stride.
int get_map(const void* ptr, long long rows, long long K, long long rs, long long ks, long long bo,
            long long bi, int hdiv, int nb, int box_rows, MapVal* out, char* err) {
  static std::unordered_map<MapKey, MapVal, MapKeyHash> cache;
  static std::mutex mu;
  MapKey key;
  memset(&key, 0, sizeof(key));
  key.ptr = ptr; key.rows = rows; key.K = K; key.rs = rs; key.ks = ks; key.bo = bo; key.bi = bi;
  key.hdiv = hdiv; key.nb = nb; key.box_rows = box_rows;
  std::lock_guard<std::mutex> lock(mu);
  auto itf = cache.find(key);
  if (itf != cache.end()) { *out = itf->second; return 0; }
  EncodeTiledFn enc = get_encode();
  if (!enc) { snprintf(err, 256, "gemm: cuTensorMapEncodeTiled is not available"); return MSLT_ERR_CUDA; }
  const bool mn = rs == 1 && ks != 1;
  // logical dims after dim 0: 0 = the other matrix index, 1 = inner batch, 2 = outer batch
  long long ext[3] = {mn ? K : rows, hdiv, nb};
  long long str[3] = {mn ? ks : rs, bi, bo};
  unsigned box[3] = {(unsigned)(mn ? 64 : box_rows), 1, 1};
  const long long ext0 = mn ? rows : K;
  const long long big = (long long)1 << 38;
  for (int i = 0; i < 3; i++)
    if (ext[i] == 1 && (i > 0)) str[i] = 0;
  // dims of extent 1 get a harmless stride at the end of the order
  int order[3] = {0, 1, 2};
  auto eff = [&](int i) { return (ext[i] == 1 && i > 0) ? big : str[i]; };
  for (int i = 0; i < 3; i++)
    for (int j = i + 1; j < 3; j++)
      if (eff(order[j]) < eff(order[i])) { int t = order[i]; order[i] = order[j]; order[j] = t; }
  cuuint64_t gdim[4], gstr[3];
  cuuint32_t bdim[4], estr[4] = {1, 1, 1, 1};
  gdim[0] = (cuuint64_t)ext0;
  bdim[0] = 64;
  long long last = 16;
  for (int sl = 0; sl < 3; sl++) {
    const int li = order[sl];
    gdim[sl + 1] = (cuuint64_t)ext[li];
    bdim[sl + 1] = box[li];
    long long sb = eff(li) == big ? last : str[li] * 2;
    if (sb <= 0 || sb % 16) {
      snprintf(err, 256, "gemm: operand stride %lld bytes is not a positive multiple of 16", sb);
      return MSLT_ERR_ARG;
    }
    gstr[sl] = (cuuint64_t)sb;
    last = sb * (long long)ext[li];
    out->perm[li] = sl + 1;
  }
  if ((uintptr_t)ptr & 15) { snprintf(err, 256, "gemm: operand base is not 16-byte aligned"); return MSLT_ERR_ARG; }
  CUresult r = enc(&out->map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), gdim, gstr, bdim,
                   estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(err, 256, "gemm: cuTensorMapEncodeTiled failed with code %d (dims %llu,%llu,%llu,%llu)", (int)r,
             (unsigned long long)gdim[0], (unsigned long long)gdim[1], (unsigned long long)gdim[2],
             (unsigned long long)gdim[3]);
    return MSLT_ERR_CUDA;
  }
  if (cache.size() > 4096) cache.clear();
  cache[key] = *out;
  return 0;
}

}  // namespace
}  // namespace mslt
