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
#include "ptx.cuh"

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
  float* rowstat;     // [units][kHeadStatFloats], first 8 of a unit: the heads' log-sum-exp (log2 domain), left for the post-eviction output; may be null
  int stat_tag;       // what the plan kernel writes into the workspace header's statistics tag; < 0: leaves it alone
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
  pl.rowstat = nullptr;
  pl.stat_tag = kStatNone;
  if (out) *out = pl;
  return off;
}

// ---- plan: items per unit, their prefix sum, and cleared counters / flags (one CTA) -------------
__global__ void __launch_bounds__(1024)
plan_kernel(int units, int Hkv, int cap, const int* __restrict__ len, Plan pl, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  __shared__ int warp_tot[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) {
    carry = 0; pl.item_prefix[0] = 0; pl.work[0] = 0; pl.work[1] = 0;
    if (pl.stat_tag >= 0) status[kStatTagIndex] = pl.stat_tag;
  }
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

// ---- PTX wrappers (ptx.cuh) and the waits built on them --------------------------------------------------
using ptx::smem_u32;
using ptx::mbar_init;
using ptx::mbar_expect_tx;
using ptx::mbar_arrive;
using ptx::mbar_try_wait;
using ptx::policy_evict_first;
using ptx::policy_evict_last;
using ptx::tma_load_2d;
using ptx::bulk_load;
using ptx::fence_async_smem;
using ptx::fence_async_all;
using ptx::fast_exp2;
using ptx::tile_off;

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
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
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



}  // namespace decode
}  // namespace caote
