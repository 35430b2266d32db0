// Single-query (decode) scoring path for bf16, head_dim 128, group size <= 8: one persistent kernel
// that reads K and V from HBM once and takes the second pass over V out of L2.
//
// Work list. A unit's cached tokens are cut into tiles of kT tokens and items of `tpi` consecutive
// tiles. Every item appears twice in one global, statically ordered work list:
//   A(i)  attention pass: logits of the G group heads (tensor cores, mma.sync bf16), online softmax
//         over the item's tiles, partial output sum_j p_j v_j; the logits go to a scratch array, the
//         (max, sum, partial output) record to another; the CTA that completes a unit's last A item
//         merges the records into the final softmax statistics, the attention output o and the
//         reference vector X, and raises the unit's ready flag;
//   B(i)  score pass: re-reads the item's V tiles (still in L2: B(i) trails A(i) by `lag` items, a few
//         tens of MB) and its logits, and writes c_j = w_j / (1 - w_j) * ||X - v_j|| once.
// The list is A(0..lag-1), then B(0), A(lag), B(1), A(lag+1), ..., then the remaining B items. CTAs
// take entries with one atomic counter, so a CTA that is busy merging simply takes fewer entries.
//
// Inside a CTA one producer warp walks the work list and fills a ring of shared-memory slots by TMA
// (a K tile, a V tile, or a V tile plus the tile's logits and carried base scores); eight consumer
// warps process the slots in order. Full/empty mbarriers hand the slots back and forth.
//
// Waits. B(i) needs its unit's ready flag. `lag` is at least the number of items of the longest
// unit, so every A item of that unit was taken from the list before B(i) was, by a CTA that is
// running and that only has earlier list entries in front of it; by induction over the list order
// every flag is raised. No co-residency of the whole grid is needed. Every wait is still bounded by a
// clock limit; when one runs out the CTA records CAOTE_ERR_TIMEOUT, stops taking work, lets its own
// copies land and returns.
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
constexpr int kSlots = 3;
constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kThreads = kConsumers + 32;  // + one producer warp
constexpr int kHalfBytes = kT * 128;       // one 64-channel box: kT rows of 128 bytes
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kRowsBytes = 8 * kT * 4;     // per slot: 8 rows of kT floats (logits / base / q / P fragments)
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
constexpr int kSideBytes = kRowsBytes + kFinalBytes;   // the rows, then the unit's FinalRec (score-pass slots)

struct Desc {         // what a slot holds
  int type, unit, tile, n_valid, flags, item, item0, nitems;
};

struct Plan {
  int* item_prefix;   // [units + 1] exclusive prefix of items per unit
  int* counter;       // [units] A items of the unit whose records are written
  int* ready;         // [units] 1 once FinalRec is written
  int* work;          // [1] next entry of the work list
  PartialRec* part;   // [max items]
  FinalRec* fin;      // [units]
  float* S;           // [units][G][capS] log2-domain logits
  int tpi;            // tiles per item
  int capS;           // cap rounded up to a multiple of kT
  int lag;            // items by which the score pass trails the attention pass
};

inline int tiles_per_item(const Dims& dm, int grid) {
  const long long max_tiles = (long long)dm.units * ((dm.cap + kT - 1) / kT);
  long long t = max_tiles / (2LL * (grid > 0 ? grid : 1));
  if (t < 1) t = 1;
  if (t > kMaxTilesPerItem) t = kMaxTilesPerItem;
  return (int)t;
}

// `grid` only shapes the item size and the lag; the carve must be called with the same value by
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
  pl.lag = (tiles_per_unit + pl.tpi - 1) / pl.tpi + (grid > 0 ? grid : 1);
  const size_t max_items = (size_t)dm.units * tiles_per_unit;  // sized for tpi = 1
  pl.item_prefix = (int*)take(sizeof(int) * ((size_t)dm.units + 1));
  pl.counter = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.ready = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.work = (int*)take(sizeof(int) * 4);
  pl.fin = (FinalRec*)take(sizeof(FinalRec) * (size_t)dm.units);
  pl.S = (float*)take(sizeof(float) * (size_t)dm.units * dm.G * pl.capS);
  pl.part = (PartialRec*)take(sizeof(PartialRec) * max_items);
  if (out) *out = pl;
  return off;
}

inline size_t smem_bytes() {
  return 1024 /* alignment slack */ + (size_t)kSlots * (kTileBytes + kSideBytes) + sizeof(Desc) * kSlots +
         sizeof(float) * (2 * kConsumerWarps * 8 + kConsumerWarps * 8 + kConsumerWarps + 8 + kD) + 8 * 2 * kSlots + 64;
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
    if (u < units) pl.item_prefix[u + 1] = before + incl;
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
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Barrier of the consumer warps only (the producer warp never joins it).
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }
// The same barrier with an OR-reduction: every consumer thread gets the same answer.
__device__ __forceinline__ bool consumer_any(bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.or.pred q, 1, %2, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"((uint32_t)pred), "n"(kConsumers)
      : "memory");
  return r != 0;
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Two floats -> packed bf16x2 (x0 in the low half), round to nearest even.
__device__ __forceinline__ uint32_t pack_bf16(float x0, float x1) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x1), "f"(x0));
  return r;
}
// bf16 hi/lo split of two floats: x ~= hi + lo with ~16 significant bits.
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  hi = pack_bf16(x0, x1);
  lo = pack_bf16(x0 - __uint_as_float(hi << 16), x1 - __uint_as_float(hi & 0xffff0000u));
}
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

// Entry w of the work list -> (is_B, item). N items, lag L (see the file comment).
__device__ __forceinline__ void work_entry(int w, int N, int L, bool& is_b, int& item) {
  if (L > N) L = N;
  if (w < L) { is_b = false; item = w; return; }
  if (w < 2 * N - L) {
    const int r = w - L;
    is_b = (r & 1) == 0;
    item = is_b ? (r >> 1) : (L + (r >> 1));
    return;
  }
  is_b = true;
  item = w - N;
}

__global__ void __launch_bounds__(kThreads, 2)
decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, Dims dm,
              const __nv_bfloat16* __restrict__ q, const int* __restrict__ len, float* __restrict__ base,
              float* __restrict__ o, float* __restrict__ scores, Plan pl, int* status) {
  extern __shared__ char smem_raw[];
  char* sm = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  char* tiles = sm;                                                              // [kSlots][kTileBytes]
  char* sides = tiles + kSlots * kTileBytes;                                     // [kSlots][kSideBytes]
  Desc* desc = reinterpret_cast<Desc*>(sides + kSlots * kSideBytes);             // [kSlots]
  float* wmax = reinterpret_cast<float*>(desc + kSlots);                         // [2][kConsumerWarps][8]
  float* wl = wmax + 2 * kConsumerWarps * 8;                                     // [kConsumerWarps][8]
  float* whb = wl + kConsumerWarps * 8;                                          // [kConsumerWarps]
  float* wm = whb + kConsumerWarps;                                              // [8]
  float* xrow = wm + 8;                                                          // [kD]
  uint64_t* full = reinterpret_cast<uint64_t*>(xrow + kD);                       // [kSlots]
  uint64_t* empty = full + kSlots;                                               // [kSlots]
  volatile int* ctl = reinterpret_cast<volatile int*>(empty + kSlots);           // [0] stop, [1] last arriver,
                                                                                 // [2] slots issued

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = dm.G, mode = dm.base_mode;
  const bool use_base = (mode == CAOTE_BASE_ACCUM || mode == CAOTE_BASE_EXTERNAL);
  const bool softmax_counted = (mode != CAOTE_BASE_EXTERNAL);
  const float scale2 = dm.scale * 1.4426950408889634f;  // logits are kept in the log2 domain
  const int N = pl.item_prefix[dm.units];

  if (tid == 0) {
    for (int i = 0; i < kSlots; ++i) {
      mbar_init(&full[i], 1);
      mbar_init(&empty[i], kConsumerWarps);
    }
    ctl[0] = 0;
    ctl[1] = 0;
    ctl[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kSlots * (int)(sizeof(Desc) / sizeof(int))) reinterpret_cast<int*>(desc)[tid] = 0;
  __syncthreads();

  int consumed = 0;  // slots the consumers have finished (uniform over the consumer threads)

  if (warp == kConsumerWarps) {
    // ================================ producer warp ================================
    const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
    int issued = 0;
    bool ok = true;
    auto acquire_slot = [&](int& s) -> bool {  // lane 0
      s = issued % kSlots;
      return mbar_wait(&empty[s], ((issued / kSlots) & 1) ^ 1, &ctl[0]);
    };
    while (ok) {
      int w = 0;
      if (lane == 0) w = atomicAdd(pl.work, 1);
      w = __shfl_sync(0xffffffffu, w, 0);
      if (w >= 2 * N) break;
      bool is_b;
      int item;
      work_entry(w, N, pl.lag, is_b, item);
      // unit of the item: 32-ary search over the item prefix, one probe per lane
      int lo = 0, hi = dm.units;
      while (hi - lo > 1) {
        const int step = (hi - lo + 31) / 32;
        const int probe = lo + lane * step;
        const int val = (probe < hi) ? __ldg(pl.item_prefix + probe) : 0x7fffffff;
        const unsigned mask = __ballot_sync(0xffffffffu, val <= item);
        const int k = 31 - __clz((int)mask);
        lo = lo + k * step;
        hi = min(hi, lo + step);
      }
      const int u = lo;
      if (lane == 0) {
        const int item0 = pl.item_prefix[u], nitems = pl.item_prefix[u + 1] - item0;
        const int n = len[u / dm.Hkv];
        const int ntiles = (n + kT - 1) / kT;
        const int t_begin = (item - item0) * pl.tpi, t_end = min(t_begin + pl.tpi, ntiles);
        if (is_b) {
          // the item's logits and the unit's final record must be complete before they are copied
          const long long t0c = clock64();
          while (ld_acquire(&pl.ready[u]) == 0) {
            if (ctl[0] || clock64() - t0c > kWaitCycles) { ok = false; break; }
            __nanosleep(64);
          }
          fence_async_all();
        }
        for (int t = t_begin; ok && t < t_end; ++t) {
          Desc d;
          d.unit = u;
          d.tile = t;
          d.n_valid = min(kT, n - t * kT);
          d.flags = (t == t_begin ? kFlagFirst : 0) | (t == t_end - 1 ? kFlagLast : 0);
          d.item = item;
          d.item0 = item0;
          d.nitems = nitems;
          const int row = u * dm.cap + t * kT;
          const uint32_t base_bytes = use_base ? (uint32_t)min(kT, dm.cap - t * kT) * 4u : 0u;
          const float* base_src = use_base ? base + (size_t)u * dm.cap + t * kT : nullptr;
          int s;
          if (!is_b) {
            if (!(ok = acquire_slot(s))) break;
            char* tl = tiles + s * kTileBytes;
            char* sd = sides + s * kSideBytes;
            d.type = kSlotKA;
            desc[s] = d;
            // the unit's G query rows ride along with the item's first K tile (rows 0..3 of the side area)
            const uint32_t q_bytes = (d.flags & kFlagFirst) ? (uint32_t)G * kD * 2u : 0u;
            mbar_expect_tx(&full[s], kTileBytes + base_bytes + q_bytes);
            tma_load_2d(tl, &tmK, 0, row, &full[s], pol_stream);
            tma_load_2d(tl + kHalfBytes, &tmK, 64, row, &full[s], pol_stream);
            if (use_base) bulk_load(sd + 7 * kT * 4, base_src, base_bytes, &full[s]);
            if (q_bytes)
              bulk_load(sd, q + ((size_t)(u / dm.Hkv) * dm.Hq + (size_t)(u % dm.Hkv) * G) * kD, q_bytes, &full[s]);
            ctl[2] = ++issued;
            if (!(ok = acquire_slot(s))) break;
            tl = tiles + s * kTileBytes;
            d.type = kSlotVA;
            desc[s] = d;
            mbar_expect_tx(&full[s], kTileBytes);
            tma_load_2d(tl, &tmV, 0, row, &full[s], pol_keep);
            tma_load_2d(tl + kHalfBytes, &tmV, 64, row, &full[s], pol_keep);
            ctl[2] = ++issued;
          } else {
            if (!(ok = acquire_slot(s))) break;
            char* tl = tiles + s * kTileBytes;
            char* sd = sides + s * kSideBytes;
            d.type = kSlotVB;
            desc[s] = d;
            const uint32_t s_bytes = softmax_counted ? (uint32_t)G * kT * 4u : 0u;
            mbar_expect_tx(&full[s], kTileBytes + s_bytes + base_bytes + kFinalBytes);
            tma_load_2d(tl, &tmV, 0, row, &full[s], pol_stream);
            tma_load_2d(tl + kHalfBytes, &tmV, 64, row, &full[s], pol_stream);
            if (softmax_counted) {
              const float* ssrc = pl.S + ((size_t)u * G) * pl.capS + (size_t)t * kT;
              for (int g = 0; g < G; ++g)
                bulk_load(sd + g * kT * 4, ssrc + (size_t)g * pl.capS, kT * 4, &full[s]);
            }
            if (use_base) bulk_load(sd + 7 * kT * 4, base_src, base_bytes, &full[s]);
            bulk_load(sd + kRowsBytes, pl.fin + u, kFinalBytes, &full[s]);
            ctl[2] = ++issued;
          }
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    if (lane == 0) {
      if (ok) {
        int s;
        if (acquire_slot(s)) {
          desc[s].type = kSlotStop;
          mbar_arrive(&full[s]);
          ctl[2] = ++issued;
        } else {
          ok = false;
        }
      }
      if (!ok && !ctl[0]) {  // a wait of the producer's own ran out
        set_status(status, CAOTE_ERR_TIMEOUT);
        ctl[0] = 1;
      }
    }
  } else {
    // ================================ consumer warps ================================
    const int head = lane >> 2, quad = lane & 3;
    const int t0 = 16 * warp + 2 * quad;  // this thread's tokens: t0, t0 + 1, t0 + 8, t0 + 9
    uint32_t qa[8][2];
    float m_run = -INFINITY, l_priv = 0.f, hb_priv = 0.f, corr = 0.f;
    float o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
    int tile_par = 0;

    for (;; ++consumed) {
      const int s = consumed % kSlots;
      char* sl = tiles + s * kTileBytes;
      float* side = reinterpret_cast<float*>(sides + s * kSideBytes);  // [8][kT], then a FinalRec
      const bool got = warp_mbar_wait(&full[s], (consumed / kSlots) & 1, &ctl[0], lane);
      if (consumer_any(!got)) {  // uniform: either every consumer thread leaves here or none does
        if (tid == 0 && !ctl[0]) {
          set_status(status, CAOTE_ERR_TIMEOUT);
          ctl[0] = 1;
        }
        break;
      }
      const Desc d = desc[s];
      if (d.type == kSlotStop) { ++consumed; break; }
      const int b = d.unit / dm.Hkv, h = d.unit % dm.Hkv;

      if (d.type == kSlotKA) {
        // ===================== logits and softmax numerators of one tile =====================
        if (d.flags & kFlagFirst) {
          // Q fragments: row = lane / 4 (rows 8..15 duplicate rows 0..7), zero for heads >= G
          const __nv_bfloat16* qrow = reinterpret_cast<const __nv_bfloat16*>(side) + (head < G ? head : 0) * kD + 2 * quad;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = (head < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks) : 0u;
            qa[ks][1] = (head < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8) : 0u;
          }
          m_run = -INFINITY;
          l_priv = 0.f;
          hb_priv = 0.f;
#pragma unroll
          for (int i = 0; i < 4; ++i) { o0[i] = 0.f; o1[i] = 0.f; }
        }
        const uint32_t kaddr = smem_u32(sl);
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
          const int mi = lane >> 3, r = lane & 7;
          const int tok = 16 * warp + 8 * (mi >> 1) + r;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(kaddr + tile_off(tok, 2 * ks + (mi & 1)), b0, b1, b2, b3);
            mma_bf16(s0, qa[ks][0], qa[ks][0], qa[ks][1], qa[ks][1], b0, b1);
            mma_bf16(s1, qa[ks][0], qa[ks][0], qa[ks][1], qa[ks][1], b2, b3);
          }
        }
        const bool v0 = t0 < d.n_valid, v1 = t0 + 1 < d.n_valid, v2 = t0 + 8 < d.n_valid, v3 = t0 + 9 < d.n_valid;
        float bv[4] = {0.f, 0.f, 0.f, 0.f};
        if (use_base && head == 7) {
          const float* Bb = side + 7 * kT;
          bv[0] = v0 ? Bb[t0] : 0.f;
          bv[1] = v1 ? Bb[t0 + 1] : 0.f;
          bv[2] = v2 ? Bb[t0 + 8] : 0.f;
          bv[3] = v3 ? Bb[t0 + 9] : 0.f;
          hb_priv += (bv[0] + bv[1]) + (bv[2] + bv[3]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);  // this warp is done with the K tile and its base row

        float sv[4];
        sv[0] = v0 ? s0[0] * scale2 : -INFINITY;
        sv[1] = v1 ? s0[1] * scale2 : -INFINITY;
        sv[2] = v2 ? s1[0] * scale2 : -INFINITY;
        sv[3] = v3 ? s1[1] * scale2 : -INFINITY;
        if (softmax_counted && head < G) {
          float* Sg = pl.S + ((size_t)d.unit * G + head) * pl.capS + (size_t)d.tile * kT + t0;
          __stcg(reinterpret_cast<float2*>(Sg), make_float2(sv[0], sv[1]));
          __stcg(reinterpret_cast<float2*>(Sg + 8), make_float2(sv[2], sv[3]));
        }
        float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
        float* wmx = wmax + tile_par * kConsumerWarps * 8;
        if (quad == 0) wmx[warp * 8 + head] = mx;
        consumer_sync();
        float m_new = m_run;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) m_new = fmaxf(m_new, wmx[w * 8 + head]);
        tile_par ^= 1;
        corr = fast_exp2(m_run - m_new);  // m_new is finite (a tile holds a valid token); 2^-inf = 0
        m_run = m_new;
        float p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = fast_exp2(sv[i] - m_new);
        l_priv = fmaf(l_priv, corr, (p[0] + p[1]) + (p[2] + p[3]));
        if (head >= G) { p[0] = p[1] = p[2] = p[3] = 0.f; }
        if (use_base && head == 7) {
          p[0] = bv[0]; p[1] = bv[1]; p[2] = bv[2]; p[3] = bv[3];
          corr = 1.f;
        }
        uint4 frag;  // a0 = hi(n-tile 0), a1 = lo(n-tile 0), a2 = hi(n-tile 1), a3 = lo(n-tile 1)
        split_pair(p[0], p[1], frag.x, frag.y);
        split_pair(p[2], p[3], frag.z, frag.w);
        // the P fragments wait in the side area of the next slot, which will hold this tile's V
        uint4* Pbuf = reinterpret_cast<uint4*>(sides + ((consumed + 1) % kSlots) * kSideBytes);
        Pbuf[warp * 32 + lane] = frag;
      } else if (d.type == kSlotVA) {
        // ===================== partial output of one tile =====================
        const uint4* Pbuf = reinterpret_cast<const uint4*>(side);
        if (d.n_valid < kT) {
          // rows behind the unit's length hold whatever the cache has there: clear them so that a
          // zero weight times a stray NaN cannot reach the accumulators
          const int rows = kT - d.n_valid;
          for (int i = tid; i < rows * 16; i += kConsumers) {
            const int row = d.n_valid + (i >> 4), c = i & 15;
            *reinterpret_cast<uint4*>(sl + tile_off(row, c)) = make_uint4(0u, 0u, 0u, 0u);
          }
          consumer_sync();
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) { o0[i] *= corr; o1[i] *= corr; }
        const uint32_t vaddr = smem_u32(sl);
        {
          const int mi = lane >> 3, r = lane & 7;
#pragma unroll
          for (int kk = 0; kk < kT / 16; ++kk) {
            const uint4 a = Pbuf[kk * 32 + lane];
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4_trans(vaddr + tile_off(16 * kk + 8 * (mi & 1) + r, 2 * warp + (mi >> 1)), b0, b1, b2, b3);
            mma_bf16(o0, a.x, a.y, a.z, a.w, b0, b1);
            mma_bf16(o1, a.x, a.y, a.z, a.w, b2, b3);
          }
        }
        __syncwarp();
        fence_async_smem();
        if (lane == 0) mbar_arrive(&empty[s]);

        if (d.flags & kFlagLast) {
          // ---------- the item's record ----------
          PartialRec* pr = pl.part + d.item;
          {
            const int c0 = 16 * warp + 2 * quad;
            *reinterpret_cast<float2*>(&pr->o[head][c0]) = make_float2(o0[0] + o0[2], o0[1] + o0[3]);
            *reinterpret_cast<float2*>(&pr->o[head][c0 + 8]) = make_float2(o1[0] + o1[2], o1[1] + o1[3]);
          }
          float ls = l_priv;
          ls += __shfl_xor_sync(0xffffffffu, ls, 1);
          ls += __shfl_xor_sync(0xffffffffu, ls, 2);
          float hs = hb_priv;
          hs += __shfl_xor_sync(0xffffffffu, hs, 1);
          hs += __shfl_xor_sync(0xffffffffu, hs, 2);
          if (quad == 0) {
            wl[warp * 8 + head] = ls;
            if (head == 7) whb[warp] = hs;
            if (warp == 0) wm[head] = m_run;
          }
          consumer_sync();
          if (warp == 0) {
            if (lane < 8) {
              float ll = 0.f;
              for (int w = 0; w < kConsumerWarps; ++w) ll += wl[w * 8 + lane];
              pr->m[lane] = wm[lane];
              pr->l[lane] = ll;
            }
            if (lane == 8) {
              float hb = 0.f;
              for (int w = 0; w < kConsumerWarps; ++w) hb += whb[w];
              pr->hb = use_base ? hb : 0.f;
            }
          }
          consumer_sync();
          if (tid == 0) {
            __threadfence();
            const int old = atomicAdd(&pl.counter[d.unit], 1);
            ctl[1] = (old == d.nitems - 1);
          }
          consumer_sync();
          if (ctl[1]) {
            // ---------- last arriver: merge the unit's records ----------
            __threadfence();
            const PartialRec* p0 = pl.part + d.item0;
            const int hd = tid >> 5, c4 = (tid & 31) * 4;
            const bool base_row = use_base && hd == 7;
            float mfin = -INFINITY;
            for (int c = 0; c < d.nitems; ++c) mfin = fmaxf(mfin, __ldcg(&p0[c].m[hd]));
            float lfin = 0.f, hbsum = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 4
            for (int c = 0; c < d.nitems; ++c) {
              const float f = base_row ? 1.f : exp2f(__ldcg(&p0[c].m[hd]) - mfin);
              lfin = fmaf(__ldcg(&p0[c].l[hd]), f, lfin);
              const float4 v = __ldcg(reinterpret_cast<const float4*>(&p0[c].o[hd][c4]));
              acc.x = fmaf(v.x, f, acc.x);
              acc.y = fmaf(v.y, f, acc.y);
              acc.z = fmaf(v.z, f, acc.z);
              acc.w = fmaf(v.w, f, acc.w);
              hbsum += __ldcg(&p0[c].hb);
            }
            const float inv_l = (hd < G) ? 1.f / lfin : 0.f;
            FinalRec* fr = pl.fin + d.unit;
            float4 contrib = make_float4(0.f, 0.f, 0.f, 0.f);
            if (hd < G) {
              const float4 on = make_float4(acc.x * inv_l, acc.y * inv_l, acc.z * inv_l, acc.w * inv_l);
              *reinterpret_cast<float4*>(o + ((size_t)b * dm.Hq + h * G + hd) * kD + c4) = on;
              if (softmax_counted) contrib = on;
            } else if (base_row) {
              contrib = acc;
            }
            const float Htot = (softmax_counted ? (float)G : 0.f) + (use_base ? hbsum : 0.f);
            // X = (sum of the 8 rows of contrib) / Htot; row hd lives in warp hd, so the warps add
            // their rows one after the other (fixed order: bit-reproducible)
            for (int r = 0; r < 8; ++r) {
              if (hd == r) {
                float4* xp = reinterpret_cast<float4*>(&xrow[c4]);
                float4 t = (r == 0) ? make_float4(0.f, 0.f, 0.f, 0.f) : *xp;
                t.x += contrib.x; t.y += contrib.y; t.z += contrib.z; t.w += contrib.w;
                *xp = t;
              }
              consumer_sync();
            }
            if ((tid & 31) == 0) { fr->m[hd] = mfin; fr->inv_l[hd] = inv_l; }
            if (tid == 0) fr->H = Htot;
            if (tid < kD) {
              const float xv = (Htot > 0.f) ? xrow[tid] / Htot : 0.f;
              fr->X[tid] = xv;
              float xx = warp_sum(xv * xv);
              if (lane == 0) wl[warp] = xx;  // warps 0..3
            }
            consumer_sync();
            if (tid == 0) fr->XX = (wl[0] + wl[1]) + (wl[2] + wl[3]);
            if (tid == 0) {
              __threadfence();
              st_release(&pl.ready[d.unit], 1);
            }
          }
        }
      } else {
        // ===================== score pass of one tile =====================
        // ||X - v_j||^2 = ||v_j||^2 - 2 <v_j, X> + ||X||^2 for this warp's 16 tokens on the tensor
        // cores: the V rows are the A operand; used again as the B operand they give the Gram
        // blocks whose diagonals are ||v_j||^2; X, split into bf16 hi + lo columns, gives <v_j, X>.
        // Tokens for which that difference cancels (v_j close to X) or that hold most of the weight
        // are redone below by plain subtraction, so v_j = X still scores exactly 0.
        const FinalRec* fr = reinterpret_cast<const FinalRec*>(side + 8 * kT);
        uint32_t xb[8][2];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          xb[ks][0] = 0u;
          xb[ks][1] = 0u;
          if (head < 2) {
            const float2 x0 = *reinterpret_cast<const float2*>(fr->X + 16 * ks + 2 * quad);
            const float2 x1 = *reinterpret_cast<const float2*>(fr->X + 16 * ks + 8 + 2 * quad);
            uint32_t h0, l0, h1, l1;
            split_pair(x0.x, x0.y, h0, l0);
            split_pair(x1.x, x1.y, h1, l1);
            xb[ks][0] = head == 0 ? h0 : l0;
            xb[ks][1] = head == 0 ? h1 : l1;
          }
        }
        float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f}, cx[4] = {0.f, 0.f, 0.f, 0.f};
        {
          const uint32_t vaddr = smem_u32(sl);
          const int mi = lane >> 3, r = lane & 7;
          const int tok = 16 * warp + 8 * (mi & 1) + r;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(vaddr + tile_off(tok, 2 * ks + (mi >> 1)), a0, a1, a2, a3);
            mma_bf16(ca, a0, a1, a2, a3, a0, a2);  // rows x tokens 0..7 of the warp
            mma_bf16(cb, a0, a1, a2, a3, a1, a3);  // rows x tokens 8..15
            mma_bf16(cx, a0, a1, a2, a3, xb[ks][0], xb[ks][1]);
          }
        }
        // lane (head, quad): token `head` of the warp if quad == 0, token head + 8 if quad == 1
        const int src = (lane & ~3) | (head >> 1);
        const float vva = __shfl_sync(0xffffffffu, (head & 1) ? ca[1] : ca[0], src);
        const float vvb = __shfl_sync(0xffffffffu, (head & 1) ? cb[3] : cb[2], src);
        const float vxa = __shfl_sync(0xffffffffu, cx[0] + cx[1], lane & ~3);
        const float vxb = __shfl_sync(0xffffffffu, cx[2] + cx[3], lane & ~3);
        // base score: heads quad and quad + 4 of both tokens, then a sum over the quad
        const int ra = 16 * warp + head, rb = ra + 8;
        float ha = 0.f, hbv = 0.f;
        if (softmax_counted) {
#pragma unroll
          for (int gg = 0; gg < 2; ++gg) {
            const int g = quad + 4 * gg;
            if (g < G) {
              const float mg = fr->m[g], il = fr->inv_l[g];
              ha = fmaf(fast_exp2(side[g * kT + ra] - mg), il, ha);
              hbv = fmaf(fast_exp2(side[g * kT + rb] - mg), il, hbv);
            }
          }
          ha += __shfl_xor_sync(0xffffffffu, ha, 1);
          ha += __shfl_xor_sync(0xffffffffu, ha, 2);
          hbv += __shfl_xor_sync(0xffffffffu, hbv, 1);
          hbv += __shfl_xor_sync(0xffffffffu, hbv, 2);
        }
        const int row = quad == 0 ? ra : rb;
        const bool mine = quad < 2 && row < d.n_valid;
        float hj = quad == 0 ? ha : hbv;
        const float vv = quad == 0 ? vva : vvb, vx = quad == 0 ? vxa : vxb;
        const size_t slot = (size_t)d.unit * dm.cap + (size_t)d.tile * kT + row;
        if (mine) {
          if (mode == CAOTE_BASE_ACCUM) {
            hj += side[7 * kT + row];
            base[slot] = hj;
          } else if (mode == CAOTE_BASE_EXTERNAL) {
            hj = side[7 * kT + row];
          }
        }
        const float Htot = fr->H, XX = fr->XX;
        float n2 = fmaxf(vv - 2.f * vx + XX, 0.f);
        const bool redo = mine && (n2 < 2e-3f * (vv + XX) || 2.f * hj > Htot);
        unsigned todo = __ballot_sync(0xffffffffu, redo);
        while (todo) {
          const int l = __ffs((int)todo) - 1;
          todo &= todo - 1;
          const int rr = 16 * warp + (l >> 2) + 8 * (l & 3);  // the row lane l is responsible for
          const uint2 raw = *reinterpret_cast<const uint2*>(sl + tile_off(rr, lane >> 1) + (lane & 1) * 8);
          const float4 xv = *reinterpret_cast<const float4*>(fr->X + 4 * lane);
          const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
          const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
          const float d0 = xv.x - f0.x, d1 = xv.y - f0.y, d2 = xv.z - f1.x, d3 = xv.w - f1.y;
          const float exact = warp_sum(fmaf(d0, d0, d1 * d1) + fmaf(d2, d2, d3 * d3));
          if (lane == l) n2 = exact;
        }
        if (mine) {
          float ratio = 0.f;
          if (Htot > 0.f) {
            const float rest = Htot - hj;
            ratio = (rest > 0.f) ? hj / rest : INFINITY;
          }
          scores[slot] = (ratio == 0.f) ? 0.f : ((ratio == INFINITY) ? INFINITY : ratio * sqrtf(n2));
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
      }
    }
  }

  // Leave only after every copy this CTA issued has landed (bounded), whatever the reason for leaving.
  __syncthreads();
  if (tid == 0) {
    const int issued = ctl[2];
    const int dummy = 0;
    for (int j = consumed; j < issued; ++j) mbar_wait(&full[j % kSlots], (j / kSlots) & 1, &dummy);
  }
}

}  // namespace decode
}  // namespace caote
