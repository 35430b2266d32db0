// Shared by the single-query (decode) scoring path for bf16, head_dim 128, group size <= 8: the work
// plan, the records through which CTAs hand partial results to one another, and the PTX wrappers.
//
// Work items. A unit's cached tokens are cut into tiles of kT tokens and items of `tpi` consecutive
// tiles. Every item is worked on twice, each time by whichever CTA takes it from an atomic counter:
//   attention pass  logits of the G group heads, softmax numerators against a running reference,
//                   partial output sum_j p_j v_j; the logits go to a scratch array, the (reference,
//                   sum, partial output) record to another; the CTA that completes a unit's last
//                   record merges them into the final softmax statistics, the attention output o and
//                   the reference vector X, and raises the unit's ready flag;
//   score pass      re-reads the item's V tiles and its logits once the flag is up and writes
//                   c_j = w_j / (1 - w_j) * ||X - v_j||.
// Attention items never wait for anything but shared-memory slots of their own CTA, so every flag is
// raised whatever the score side of any CTA is waiting for; no co-residency of the grid is needed.
// Every wait is still bounded by a clock limit; when one runs out the CTA records CAOTE_ERR_TIMEOUT,
// stops taking work, lets its own copies land and returns.
//
// For the base modes that carry a score (ACCUM, EXTERNAL; G <= 7) row 7 of the P operand carries
// base_j, which yields sum_j base_j v_j from the same tensor-core product.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace caote {
namespace decode {

constexpr int kT = 128;                 // tokens per tile
constexpr int kD = 128;
constexpr int kHalfBytes = kT * 128;       // one 64-channel box: kT rows of 128 bytes
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kMaxTilesPerItem = 16;
constexpr long long kWaitCycles = 2000000000LL;  // ~1 s: far beyond any legitimate wait

enum SlotType { kSlotKA = 0, kSlotVA = 1, kSlotVB = 2, kSlotStop = 3 };
enum { kFlagFirst = 1, kFlagLast = 2 };

struct PartialRec {   // per item
  float m[8];         // running max of the log2-domain logits per head
  float l[8];         // sum of 2^(s - m)
  float hb;           // sum of the carried base scores of the item
  float pad[7];
  float o[8][kD];     // sum_j p_j v_j per head (row 7: sum_j base_j v_j)
};
struct FinalRec {     // per unit
  float m[8];
  float inv_l[8];
  float H;            // normaliser of the base score: counted rows + sum of carried base scores
  float XX;           // ||X||^2
  float pad[2];
  float X[kD];
};
constexpr int kFinalBytes = sizeof(FinalRec);          // 592, a multiple of 16

struct Desc {         // what a slot holds
  int type, unit, tile, n_valid, flags, item, item0, nitems;
};

struct Plan {
  int* item_prefix;   // [units + 1] exclusive prefix of items per unit
  int4* item_info;    // [items] (unit, first item of the unit, items of the unit, tokens of the unit)
  int* counter;       // [units] A items of the unit whose records are written
  int* ready;         // [units] 1 once FinalRec is written
  int* work;          // [2] next attention item, next score item
  PartialRec* part;   // [max items]
  FinalRec* fin;      // [units]
  float* S;           // [units][capS / kT][G][kT] log2-domain logits, tile by tile
  float* dist;        // [units][capS] ||mean(v) - v_j|| (FastCAOTE only)
  int tpi;            // tiles per item
  int capS;           // cap rounded up to a multiple of kT
};

inline int tiles_per_item(const Dims& dm, int grid) {
  const long long max_tiles = (long long)dm.units * ((dm.cap + kT - 1) / kT);
  long long t = max_tiles / (2LL * (grid > 0 ? grid : 1));
  if (t < 1) t = 1;
  if (t > kMaxTilesPerItem) t = kMaxTilesPerItem;
  return (int)t;
}

// `grid` only shapes the item size; the carve must be called with the same value by
// caote_workspace_bytes and by the launch (both use the resident-CTA count, or 0 without a device:
// the sizes below are upper bounds for every grid because tpi >= 1).
inline size_t carve(const Dims& dm, char* base, Plan* out, int grid) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* p = base + off;
    off = align_up(off + bytes, 256);
    return p;
  };
  Plan pl;
  const int tiles_per_unit = (dm.cap + kT - 1) / kT;
  pl.tpi = tiles_per_item(dm, grid);
  pl.capS = tiles_per_unit * kT;
  const size_t max_items = (size_t)dm.units * tiles_per_unit;  // sized for tpi = 1
  pl.item_prefix = (int*)take(sizeof(int) * ((size_t)dm.units + 1));
  pl.item_info = (int4*)take(sizeof(int4) * max_items);
  pl.counter = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.ready = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.work = (int*)take(sizeof(int) * 4);
  pl.fin = (FinalRec*)take(sizeof(FinalRec) * (size_t)dm.units);
  pl.S = (float*)take(sizeof(float) * (size_t)dm.units * dm.G * pl.capS);
  pl.dist = (float*)take(sizeof(float) * (size_t)dm.units * pl.capS);
  pl.part = (PartialRec*)take(sizeof(PartialRec) * max_items);
  if (out) *out = pl;
  return off;
}

// ---- plan: items per unit, their prefix sum, and cleared counters / flags (one CTA) -------------
__global__ void __launch_bounds__(1024)
plan_kernel(int units, int Hkv, int cap, const int* __restrict__ len, Plan pl, int* status) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; pl.item_prefix[0] = 0; pl.work[0] = 0; pl.work[1] = 0; }
  __syncthreads();
  for (int u0 = 0; u0 < units; u0 += 1024) {
    const int u = u0 + tid;
    int ni = 0;
    if (u < units) {
      const int n = len[u / Hkv];
      if (n < 0 || n > cap) set_status(status, CAOTE_ERR_BAD_LENGTH);
      else ni = ((n + kT - 1) / kT + pl.tpi - 1) / pl.tpi;
      pl.counter[u] = 0;
      pl.ready[u] = 0;
    }
    int incl = ni;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    if (u < units) {
      pl.item_prefix[u + 1] = before + incl;
      // what a CTA needs to know about an item it takes, in one load
      const int first = before + incl - ni;
      const int4 info = make_int4(u, first, ni, len[u / Hkv]);
      for (int k = 0; k < ni; ++k) pl.item_info[first + k] = info;
    }
    __syncthreads();
    if (tid == 1023) carry = before + incl;
    __syncthreads();
  }
}

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; returns false when the clock limit ran out or *stop became non-zero.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const volatile int* stop) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*stop) return false;
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}
// Untiled bulk copy global -> shared; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// 2^x, hardware approximation (2 ulp); 2^-inf = 0.
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// One lane polls the barrier, the others sleep at the warp barrier; every lane then observes the
// completed phase itself (which is what makes the copied data visible to it). Warp-uniform result.
__device__ __forceinline__ bool warp_mbar_wait(uint64_t* bar, uint32_t parity, const volatile int* stop, int lane) {
  int ok = 1;
  if (lane == 0) ok = mbar_wait(bar, parity, stop) ? 1 : 0;
  ok = __shfl_sync(0xffffffffu, ok, 0);
  if (ok) ok = mbar_try_wait(bar, parity) ? 1 : 0;
  return __all_sync(0xffffffffu, ok) != 0;
}

// Byte offset of 16-byte chunk `chunk16` (0..15 along the 128 channels) of row `row` inside a staged
// tile: two 64-channel boxes, each kT rows x 128 bytes with the 128-byte swizzle (chunk ^ (row & 7)).
__device__ __forceinline__ uint32_t tile_off(int row, int chunk16) {
  return (uint32_t)((chunk16 >> 3) * kHalfBytes + row * 128 + (((chunk16 & 7) ^ (row & 7)) << 4));
}


}  // namespace decode
}  // namespace caote
