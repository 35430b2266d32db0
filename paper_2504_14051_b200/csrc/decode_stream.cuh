// Single-query (decode) scoring path for bf16, head_dim 128, group size <= 8: one persistent kernel
// that reads K and V from HBM once and takes the second pass over V out of L2.
//
// Work. A unit's cached tokens are cut into tiles of kT tokens and items of `tpi` consecutive tiles.
// Every item is processed twice:
//   A(i)  attention pass: logits of the G group heads (tensor cores, mma.sync bf16), online softmax
//         over the item's tiles, partial output sum_j p_j v_j; the logits go to a scratch array, the
//         item's (max, sum, partial output) record to another;
//   B(i)  score pass: re-reads the item's V tiles (from L2: B work of a unit becomes available as
//         soon as the unit's records are merged and is taken before any further A work) and its
//         logits, and writes c_j = w_j / (1 - w_j) * ||X - v_j|| once.
// A items are handed out in order by one atomic counter. When the last record of a unit is written,
// the CTA that wrote it merges the unit's records into the final softmax statistics, the attention
// output o and the reference vector X, and appends the unit's B items to a global queue. Nothing
// ever waits for another CTA except at the very end (A work exhausted, last merges in flight).
//
// Inside a CTA (one per SM):
//   producer warp   claims work (B first, then A) and fills a ring of shared-memory slots by TMA:
//                   a K tile (+ q, + carried base scores), a V tile, or a V tile with the tile's
//                   logits, base scores and the unit's final record;
//   8 consumer warps process the slots in order, each on its own 16 tokens of every tile, with its
//                   own softmax reference and full-width output accumulator (P never leaves the
//                   registers); at the end of an item they merge their partial results through a
//                   staging area in shared memory, one head per warp;
//   merge warp      counts finished records per unit, merges a completed unit, publishes its B items.
// Full/empty mbarriers hand slots back and forth; every wait in the kernel is bounded by a clock
// limit, after which the CTA records CAOTE_ERR_TIMEOUT, stops taking work, lets its own copies land
// and returns. No hardware barrier is used after start-up, so a warp that gives up cannot strand
// its siblings.
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
constexpr int kSlots = 4;
constexpr int kConsumerWarps = 8;
constexpr int kConsumers = kConsumerWarps * 32;
constexpr int kProducerWarp = kConsumerWarps;
constexpr int kMergeWarp = kConsumerWarps + 1;
constexpr int kThreads = kConsumers + 64;  // + producer warp + merge warp
constexpr int kHalfBytes = kT * 128;       // one 64-channel box: kT rows of 128 bytes
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kRowsBytes = 8 * kT * 4;     // per slot: 8 rows of kT floats (logits / base / q)
constexpr int kMaxTilesPerItem = 8;
constexpr int kJobs = 8;                   // mailbox entries between the consumers and the merge warp
constexpr long long kWaitCycles = 2000000000LL;  // ~1 s: far beyond any legitimate wait

enum SlotType { kSlotKA = 0, kSlotVA = 1, kSlotVB = 2, kSlotStop = 3 };
enum { kFlagFirst = 1, kFlagLast = 2 };

struct PartialRec {   // per item
  float m[8];         // reference of the log2-domain logits per head
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
  int* item_prefix;        // [units + 1] exclusive prefix of items per unit
  int* counter;            // [units] records of the unit that are written
  int* ctr;                // [0] next A item, [1] B entries claimed, [2] B entries reserved
  unsigned long long* bq;  // [max items] B queue: (unit << 32) | (item + 1), 0 = not yet written
  PartialRec* part;        // [max items]
  FinalRec* fin;           // [units]
  float* S;                // [units][G][capS] log2-domain logits
  int tpi;                 // tiles per item
  int capS;                // cap rounded up to a multiple of kT
  int max_items;
};

inline int tiles_per_item(const Dims& dm, int grid) {
  const long long max_tiles = (long long)dm.units * ((dm.cap + kT - 1) / kT);
  long long t = max_tiles / (4LL * (grid > 0 ? grid : 1));
  if (t < 1) t = 1;
  if (t > kMaxTilesPerItem) t = kMaxTilesPerItem;
  return (int)t;
}

// `grid` only shapes the item size; the sizes below hold for every grid (they assume tpi = 1).
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
  const size_t max_items = (size_t)dm.units * tiles_per_unit;
  pl.max_items = (int)max_items;
  pl.item_prefix = (int*)take(sizeof(int) * ((size_t)dm.units + 1));
  pl.counter = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.ctr = (int*)take(sizeof(int) * 4);
  pl.bq = (unsigned long long*)take(sizeof(unsigned long long) * max_items);
  pl.fin = (FinalRec*)take(sizeof(FinalRec) * (size_t)dm.units);
  pl.S = (float*)take(sizeof(float) * (size_t)dm.units * dm.G * pl.capS);
  pl.part = (PartialRec*)take(sizeof(PartialRec) * max_items);
  if (out) *out = pl;
  return off;
}

// Staging area in which the eight consumer warps put their partial results at the end of an item
// (two copies, used by alternate items): per warp 8 heads x kD floats, then reference, sum, base sum.
constexpr int kStageFloats = kConsumerWarps * 8 * kD + 2 * kConsumerWarps * 8 + kConsumerWarps;
constexpr int kStageBytes = (kStageFloats * 4 + 255) / 256 * 256;

struct Job {  // a finished record, handed to the merge warp
  int seq, unit, item0, nitems;
};

inline size_t smem_bytes() {
  return 1024 /* alignment slack */ + (size_t)kSlots * (kTileBytes + kSideBytes) + 2 * (size_t)kStageBytes +
         sizeof(Desc) * kSlots + sizeof(Job) * kJobs + 8 * (2 * kSlots + 4) + 64;
}

// ---- plan: items per unit, their prefix sum, and cleared counters and queue ----------------------
// grid = any number of CTAs of 1024 threads; CTA 0 computes the prefix, all clear the queue.
__global__ void __launch_bounds__(1024)
plan_kernel(int units, int Hkv, int cap, const int* __restrict__ len, Plan pl, int* status) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = blockIdx.x * 1024 + tid; i < pl.max_items; i += gridDim.x * 1024) pl.bq[i] = 0ull;
  if (blockIdx.x != 0) return;
  if (tid == 0) { carry = 0; pl.item_prefix[0] = 0; pl.ctr[0] = 0; pl.ctr[1] = 0; pl.ctr[2] = 0; }
  __syncthreads();
  for (int u0 = 0; u0 < units; u0 += 1024) {
    const int u = u0 + tid;
    int ni = 0;
    if (u < units) {
      const int n = len[u / Hkv];
      if (n < 0 || n > cap) set_status(status, CAOTE_ERR_BAD_LENGTH);
      else ni = ((n + kT - 1) / kT + pl.tpi - 1) / pl.tpi;
      pl.counter[u] = 0;
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

__device__ __forceinline__ int lds_acquire(const volatile int* p) {
  int v;
  asm volatile("ld.acquire.cta.shared::cta.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(const_cast<const int*>(p))) : "memory");
  return v;
}
__device__ __forceinline__ void sts_release(volatile int* p, int v) {
  asm volatile("st.release.cta.shared::cta.s32 [%0], %1;" ::"r"(smem_u32(const_cast<int*>(p))), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire64(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release64(unsigned long long* p, unsigned long long v) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, Dims dm,
              const __nv_bfloat16* __restrict__ q, const int* __restrict__ len, float* __restrict__ base,
              float* __restrict__ o, float* __restrict__ scores, Plan pl, int* status) {
  extern __shared__ char smem_raw[];
  char* sm = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  char* tiles = sm;                                                              // [kSlots][kTileBytes]
  char* sides = tiles + kSlots * kTileBytes;                                     // [kSlots][kSideBytes]
  char* stages = sides + kSlots * kSideBytes;                                    // [2][kStageBytes]
  Desc* desc = reinterpret_cast<Desc*>(stages + 2 * kStageBytes);                // [kSlots]
  Job* jobs = reinterpret_cast<Job*>(desc + kSlots);                             // [kJobs]
  uint64_t* full = reinterpret_cast<uint64_t*>(jobs + kJobs);                    // [kSlots]
  uint64_t* empty = full + kSlots;                                               // [kSlots]
  uint64_t* stage_full = empty + kSlots;                                         // [2]
  uint64_t* stage_free = stage_full + 2;                                         // [2]
  // [0] stop, [2] slots issued, [3] jobs taken by the merge warp, [4] consumer warps that have left,
  // [5] jobs posted in total, [6..7] warps that finished merging their head (per staging copy)
  volatile int* ctl = reinterpret_cast<volatile int*>(stage_free + 2);

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
    for (int i = 0; i < 2; ++i) {
      mbar_init(&stage_full[i], kConsumerWarps);
      mbar_init(&stage_free[i], kConsumerWarps);
    }
    for (int i = 0; i < 8; ++i) ctl[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < kSlots * (int)(sizeof(Desc) / sizeof(int))) reinterpret_cast<int*>(desc)[tid] = 0;
  if (tid < kJobs * (int)(sizeof(Job) / sizeof(int))) reinterpret_cast<int*>(jobs)[tid] = 0;
  __syncthreads();

  int consumed = 0;  // slots this warp has finished

  if (warp == kProducerWarp) {
    // ================================ producer warp ================================
    const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
    int issued = 0;
    bool ok = true;
    auto acquire_slot = [&](int& s) -> bool {  // lane 0
      s = issued % kSlots;
      return mbar_wait(&empty[s], ((issued / kSlots) & 1) ^ 1, &ctl[0]);
    };
    while (ok) {
      // ---- claim work: a published B item if there is one, else the next A item
      int kind = 0, item = 0, u = 0;  // kind: 0 = all work handed out, 1 = A, 2 = B, -1 = gave up
      if (lane == 0) {
        const long long t0c = clock64();
        for (;;) {
          const int bh = *reinterpret_cast<volatile int*>(&pl.ctr[1]);
          const int bt = ld_acquire(&pl.ctr[2]);
          if (bh < bt) {
            if (atomicCAS(&pl.ctr[1], bh, bh + 1) != bh) continue;
            unsigned long long e = ld_acquire64(&pl.bq[bh]);
            while (e == 0ull) {  // reserved, about to be written
              if (ctl[0] || clock64() - t0c > kWaitCycles) break;
              __nanosleep(32);
              e = ld_acquire64(&pl.bq[bh]);
            }
            if (e == 0ull) { kind = -1; break; }
            u = (int)(e >> 32);
            item = (int)(e & 0xffffffffull) - 1;
            kind = 2;
            break;
          }
          if (*reinterpret_cast<volatile int*>(&pl.ctr[0]) < N) {
            const int a = atomicAdd(&pl.ctr[0], 1);
            if (a < N) { item = a; kind = 1; break; }
          }
          if (bh >= N) { kind = 0; break; }
          if (ctl[0] || clock64() - t0c > kWaitCycles) { kind = -1; break; }
          __nanosleep(128);
        }
      }
      kind = __shfl_sync(0xffffffffu, kind, 0);
      item = __shfl_sync(0xffffffffu, item, 0);
      u = __shfl_sync(0xffffffffu, u, 0);
      if (kind <= 0) { ok = (kind == 0); break; }
      const bool is_b = kind == 2;
      if (!is_b) {
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
        u = lo;
      }
      if (lane == 0) {
        const int item0 = pl.item_prefix[u], nitems = pl.item_prefix[u + 1] - item0;
        const int n = len[u / dm.Hkv];
        const int ntiles = (n + kT - 1) / kT;
        const int t_begin = (item - item0) * pl.tpi, t_end = min(t_begin + pl.tpi, ntiles);
        if (is_b) fence_async_all();  // the logits and the final record were written by ordinary stores
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
  } else if (warp == kMergeWarp) {
    // ================================ merge warp ================================
    int idx = 0;
    long long t_idle = clock64();
    for (;;) {
      int state = 0;  // 1 = a job is waiting, 2 = all done, 3 = give up
      if (lane == 0) {
        if (lds_acquire(&jobs[idx % kJobs].seq) == idx + 1) state = 1;
        else if (lds_acquire(&ctl[4]) == kConsumerWarps && ctl[5] == idx) state = 2;
        else if (ctl[0]) state = 2;
        else if (clock64() - t_idle > kWaitCycles) state = 3;
      }
      state = __shfl_sync(0xffffffffu, state, 0);
      if (state == 2) break;
      if (state == 3) {
        if (lane == 0) { set_status(status, CAOTE_ERR_TIMEOUT); ctl[0] = 1; }
        break;
      }
      if (state == 0) { __nanosleep(100); continue; }
      const int unit = jobs[idx % kJobs].unit, item0 = jobs[idx % kJobs].item0, nitems = jobs[idx % kJobs].nitems;
      __syncwarp();
      ++idx;
      if (lane == 0) sts_release(&ctl[3], idx);  // the mailbox entry may be reused
      t_idle = clock64();
      int last_of_unit = 0;
      if (lane == 0) {
        __threadfence();
        last_of_unit = (atomicAdd(&pl.counter[unit], 1) == nitems - 1) ? 1 : 0;
        __threadfence();
      }
      last_of_unit = __shfl_sync(0xffffffffu, last_of_unit, 0);
      if (!last_of_unit) continue;

      // ---------- the unit's last record is in: merge its records (lane = 4 channels) ----------
      const PartialRec* p0 = pl.part + item0;
      const int b = unit / dm.Hkv, h = unit % dm.Hkv;
      float M[8], L[8], hbsum = 0.f;
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) { M[hh] = -INFINITY; L[hh] = 0.f; }
      for (int c0 = 0; c0 < nitems; c0 += 32) {
        const int c = c0 + lane;
        if (c < nitems) {
#pragma unroll
          for (int hh = 0; hh < 8; ++hh) M[hh] = fmaxf(M[hh], __ldcg(&p0[c].m[hh]));
        }
      }
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) M[hh] = warp_max(M[hh]);
      for (int c0 = 0; c0 < nitems; c0 += 32) {
        const int c = c0 + lane;
        if (c < nitems) {
#pragma unroll
          for (int hh = 0; hh < 8; ++hh)
            L[hh] = fmaf(__ldcg(&p0[c].l[hh]), fast_exp2(__ldcg(&p0[c].m[hh]) - M[hh]), L[hh]);
          hbsum += __ldcg(&p0[c].hb);
        }
      }
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) L[hh] = warp_sum(L[hh]);
      hbsum = warp_sum(hbsum);
      float4 acc[8];
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) acc[hh] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
      for (int c = 0; c < nitems; ++c) {
        float f[8];
        float4 v[8];
#pragma unroll
        for (int hh = 0; hh < 8; ++hh) {
          f[hh] = __ldcg(&p0[c].m[hh]);
          v[hh] = __ldcg(reinterpret_cast<const float4*>(&p0[c].o[hh][4 * lane]));
        }
#pragma unroll
        for (int hh = 0; hh < 8; ++hh) {
          const float ff = (use_base && hh == 7) ? 1.f : fast_exp2(f[hh] - M[hh]);
          acc[hh].x = fmaf(v[hh].x, ff, acc[hh].x);
          acc[hh].y = fmaf(v[hh].y, ff, acc[hh].y);
          acc[hh].z = fmaf(v[hh].z, ff, acc[hh].z);
          acc[hh].w = fmaf(v[hh].w, ff, acc[hh].w);
        }
      }
      const float Htot = (softmax_counted ? (float)G : 0.f) + (use_base ? hbsum : 0.f);
      FinalRec* fr = pl.fin + unit;
      float4 xs = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int hh = 0; hh < 8; ++hh) {
        const bool brow = use_base && hh == 7;
        float mo = 0.f, il = 0.f;
        if (brow) {
          xs.x += acc[hh].x; xs.y += acc[hh].y; xs.z += acc[hh].z; xs.w += acc[hh].w;
        } else if (hh < G) {
          mo = M[hh];
          il = 1.f / L[hh];
          const float4 on = make_float4(acc[hh].x * il, acc[hh].y * il, acc[hh].z * il, acc[hh].w * il);
          *reinterpret_cast<float4*>(o + ((size_t)b * dm.Hq + h * G + hh) * kD + 4 * lane) = on;
          if (softmax_counted) { xs.x += on.x; xs.y += on.y; xs.z += on.z; xs.w += on.w; }
        }
        if (lane == 0) { fr->m[hh] = mo; fr->inv_l[hh] = il; }
      }
      const float inv_h = (Htot > 0.f) ? 1.f / Htot : 0.f;
      const float4 X = make_float4(xs.x * inv_h, xs.y * inv_h, xs.z * inv_h, xs.w * inv_h);
      *reinterpret_cast<float4*>(&fr->X[4 * lane]) = X;
      const float xx = warp_sum(fmaf(X.x, X.x, X.y * X.y) + fmaf(X.z, X.z, X.w * X.w));
      if (lane == 0) { fr->H = Htot; fr->XX = xx; }
      // ---------- publish the unit's B items ----------
      __syncwarp();
      int first = 0;
      if (lane == 0) first = atomicAdd(&pl.ctr[2], nitems);
      first = __shfl_sync(0xffffffffu, first, 0);
      __threadfence();
      for (int k = lane; k < nitems; k += 32)
        st_release64(&pl.bq[first + k], ((unsigned long long)(unsigned)unit << 32) | (unsigned)(item0 + k + 1));
    }
  } else {
    // ================================ consumer warps ================================
    // Each warp is on its own: it owns tokens [16 warp, 16 warp + 16) of every tile, keeps its own
    // softmax reference and its own full-width output accumulator, and never waits for a sibling
    // except where the item's eight partial results are merged.
    const int head = lane >> 2, quad = lane & 3;
    const int t0 = 16 * warp + 2 * quad;  // this thread's tokens in a tile: t0, t0 + 1, t0 + 8, t0 + 9
    const int mi = lane >> 3, mr = lane & 7;
    bool alive = true;
    int items_done = 0;  // A items this warp has finished (selects the staging copy)
    int s = 0;
    Desc d;
    auto next_slot = [&]() -> bool {
      s = consumed % kSlots;
      if (!warp_mbar_wait(&full[s], (consumed / kSlots) & 1, &ctl[0], lane)) return false;
      d = desc[s];
      return true;
    };
    auto release = [&]() {
      __syncwarp();
      fence_async_smem();
      if (lane == 0) mbar_arrive(&empty[s]);
      ++consumed;
    };

    while (alive) {
      if (!next_slot()) { alive = false; break; }
      if (d.type == kSlotStop) { ++consumed; break; }

      if (d.type == kSlotKA) {
        // =============================== one A item ===============================
        const bool base_row = use_base && head == 7;
        uint32_t qa[8][2];
        float oacc[16][4];
        float m_ref = base_row ? 0.f : -INFINITY, l_priv = 0.f, hb_priv = 0.f;
#pragma unroll
        for (int j = 0; j < 16; ++j) { oacc[j][0] = 0.f; oacc[j][1] = 0.f; oacc[j][2] = 0.f; oacc[j][3] = 0.f; }
        {
          // Q fragments: row = lane / 4 (rows 8..15 duplicate rows 0..7), zero for heads >= G
          const __nv_bfloat16* qrow = reinterpret_cast<const __nv_bfloat16*>(sides + s * kSideBytes) +
                                      (head < G ? head : 0) * kD + 2 * quad;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            qa[ks][0] = (head < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks) : 0u;
            qa[ks][1] = (head < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8) : 0u;
          }
        }
        for (;;) {
          // ---------------- K tile: logits, softmax numerators ----------------
          if (d.type != kSlotKA) { alive = false; break; }
          uint4 frag;  // P as an A fragment: a0 = hi(tokens 0..7), a1 = lo(0..7), a2 = hi(8..15), a3 = lo(8..15)
          {
            const uint32_t kaddr = smem_u32(tiles + s * kTileBytes);
            const float* side = reinterpret_cast<const float*>(sides + s * kSideBytes);
            uint32_t kb[8][4];
            const int tok = 16 * warp + 8 * (mi >> 1) + mr;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              ldmatrix_x4(kaddr + tile_off(tok, 2 * ks + (mi & 1)), kb[ks][0], kb[ks][1], kb[ks][2], kb[ks][3]);
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              mma_bf16(s0, qa[ks][0], qa[ks][0], qa[ks][1], qa[ks][1], kb[ks][0], kb[ks][1]);
              mma_bf16(s1, qa[ks][0], qa[ks][0], qa[ks][1], qa[ks][1], kb[ks][2], kb[ks][3]);
            }
            const bool v0 = t0 < d.n_valid, v1 = t0 + 1 < d.n_valid, v2 = t0 + 8 < d.n_valid, v3 = t0 + 9 < d.n_valid;
            float bv[4] = {0.f, 0.f, 0.f, 0.f};
            if (base_row) {
              const float* Bb = side + 7 * kT;
              bv[0] = v0 ? Bb[t0] : 0.f;
              bv[1] = v1 ? Bb[t0 + 1] : 0.f;
              bv[2] = v2 ? Bb[t0 + 8] : 0.f;
              bv[3] = v3 ? Bb[t0 + 9] : 0.f;
              hb_priv += (bv[0] + bv[1]) + (bv[2] + bv[3]);
            }
            const int tile = d.tile, unit = d.unit;
            release();  // done with the K tile and its side rows

            float sv[4];
            sv[0] = v0 ? s0[0] * scale2 : -INFINITY;
            sv[1] = v1 ? s0[1] * scale2 : -INFINITY;
            sv[2] = v2 ? s1[0] * scale2 : -INFINITY;
            sv[3] = v3 ? s1[1] * scale2 : -INFINITY;
            if (softmax_counted && head < G) {
              float* Sg = pl.S + ((size_t)unit * G + head) * pl.capS + (size_t)tile * kT + t0;
              __stcg(reinterpret_cast<float2*>(Sg), make_float2(sv[0], sv[1]));
              __stcg(reinterpret_cast<float2*>(Sg + 8), make_float2(sv[2], sv[3]));
            }
            float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
            // The reference moves only when a logit exceeds it by more than 8 (p stays <= 256), so
            // the 64 accumulator registers are rescaled a handful of times per item, not every tile.
            const bool need = !base_row && mx > m_ref + 8.f;  // also true for the first finite maximum
            if (__any_sync(0xffffffffu, need)) {
              const float corr = need ? fast_exp2(m_ref - mx) : 1.f;
              if (need) m_ref = mx;
              l_priv *= corr;
#pragma unroll
              for (int j = 0; j < 16; ++j) { oacc[j][0] *= corr; oacc[j][1] *= corr; oacc[j][2] *= corr; oacc[j][3] *= corr; }
            }
            float p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = (sv[i] == -INFINITY) ? 0.f : fast_exp2(sv[i] - m_ref);
            l_priv += (p[0] + p[1]) + (p[2] + p[3]);
            if (head >= G) { p[0] = p[1] = p[2] = p[3] = 0.f; }
            if (base_row) { p[0] = bv[0]; p[1] = bv[1]; p[2] = bv[2]; p[3] = bv[3]; }
            split_pair(p[0], p[1], frag.x, frag.y);
            split_pair(p[2], p[3], frag.z, frag.w);
          }
          // ---------------- V tile: partial output of this warp's 16 tokens ----------------
          if (!next_slot() || d.type != kSlotVA) { alive = false; break; }
          {
            char* sl = tiles + s * kTileBytes;
            if (d.n_valid < 16 * warp + 16) {
              // rows behind the unit's length hold whatever the cache has there: clear this warp's
              // so that a zero weight times a stray NaN cannot reach the accumulators
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int row = 16 * warp + 2 * i + (lane >> 4), c = lane & 15;
                if (row >= d.n_valid) *reinterpret_cast<uint4*>(sl + tile_off(row, c)) = make_uint4(0u, 0u, 0u, 0u);
              }
              __syncwarp();
            }
            const uint32_t vaddr = smem_u32(sl);
            const int vrow = 16 * warp + 8 * (mi & 1) + mr;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t vb[4][4];
#pragma unroll
              for (int jj = 0; jj < 4; ++jj)
                ldmatrix_x4_trans(vaddr + tile_off(vrow, 2 * (4 * half + jj) + (mi >> 1)), vb[jj][0], vb[jj][1], vb[jj][2], vb[jj][3]);
#pragma unroll
              for (int jj = 0; jj < 4; ++jj) {
                mma_bf16(oacc[2 * (4 * half + jj)], frag.x, frag.y, frag.z, frag.w, vb[jj][0], vb[jj][1]);
                mma_bf16(oacc[2 * (4 * half + jj) + 1], frag.x, frag.y, frag.z, frag.w, vb[jj][2], vb[jj][3]);
              }
            }
          }
          const bool last_tile = (d.flags & kFlagLast) != 0;
          const int unit = d.unit, item = d.item, item0 = d.item0, nitems = d.nitems;
          release();
          if (!last_tile) {
            if (!next_slot()) { alive = false; break; }
            continue;
          }
          // ---------------- end of the item: merge the eight warps' partial results ----------------
          {
            const int buf = items_done & 1, use = items_done >> 1;
            float* stage = reinterpret_cast<float*>(stages + buf * kStageBytes);
            float* sm_m = stage + kConsumerWarps * 8 * kD;   // [warp][head]
            float* sm_l = sm_m + kConsumerWarps * 8;         // [warp][head]
            float* sm_hb = sm_l + kConsumerWarps * 8;        // [warp]
            // the copy was last used two items ago; every warp signals when it is done reading it
            if (use >= 1 && !warp_mbar_wait(&stage_free[buf], (use - 1) & 1, &ctl[0], lane)) { alive = false; break; }
            float* mine = stage + (warp * 8 + head) * kD;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int c = (4 * j + quad) ^ (4 * (head & 3));  // float2 slot, swizzled against bank conflicts
              *reinterpret_cast<float2*>(mine + 2 * c) = make_float2(oacc[j][0] + oacc[j][2], oacc[j][1] + oacc[j][3]);
            }
            float ls = l_priv;
            ls += __shfl_xor_sync(0xffffffffu, ls, 1);
            ls += __shfl_xor_sync(0xffffffffu, ls, 2);
            float hs = hb_priv;
            hs += __shfl_xor_sync(0xffffffffu, hs, 1);
            hs += __shfl_xor_sync(0xffffffffu, hs, 2);
            if (quad == 0) {
              sm_m[warp * 8 + head] = m_ref;
              sm_l[warp * 8 + head] = ls;
              if (head == 7) sm_hb[warp] = hs;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&stage_full[buf]);
            if (!warp_mbar_wait(&stage_full[buf], use & 1, &ctl[0], lane)) { alive = false; break; }
            // this warp merges head `warp`; lane = 4 channels
            {
              PartialRec* pr = pl.part + item;
              const int hh = warp;
              const bool brow = use_base && hh == 7;
              float mw[kConsumerWarps], M = -INFINITY;
#pragma unroll
              for (int w = 0; w < kConsumerWarps; ++w) { mw[w] = sm_m[w * 8 + hh]; M = fmaxf(M, mw[w]); }
              float L = 0.f;
              float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
              for (int w = 0; w < kConsumerWarps; ++w) {
                const float f = brow ? 1.f : fast_exp2(mw[w] - M);
                L = fmaf(sm_l[w * 8 + hh], f, L);
                const float4 v = *reinterpret_cast<const float4*>(stage + (w * 8 + hh) * kD + 2 * ((2 * lane) ^ (4 * (hh & 3))));
                acc.x = fmaf(v.x, f, acc.x);
                acc.y = fmaf(v.y, f, acc.y);
                acc.z = fmaf(v.z, f, acc.z);
                acc.w = fmaf(v.w, f, acc.w);
              }
              *reinterpret_cast<float4*>(&pr->o[hh][4 * lane]) = acc;
              if (lane == 0) { pr->m[hh] = M; pr->l[hh] = L; }
              if (hh == 7 && lane == 0) {
                float hb_tot = 0.f;
#pragma unroll
                for (int w = 0; w < kConsumerWarps; ++w) hb_tot += sm_hb[w];
                pr->hb = use_base ? hb_tot : 0.f;
              }
            }
            __syncwarp();
            int last_warp = 0;
            if (lane == 0) {
              mbar_arrive(&stage_free[buf]);
              __threadfence_block();
              last_warp = (atomicAdd_block(const_cast<int*>(&ctl[6 + buf]), 1) == kConsumerWarps - 1) ? 1 : 0;
              __threadfence_block();
              if (last_warp) {
                // the record is complete: hand it to the merge warp
                ctl[6 + buf] = 0;
                const long long t0c = clock64();
                while (items_done - lds_acquire(&ctl[3]) >= kJobs) {
                  if (ctl[0] || clock64() - t0c > kWaitCycles) { last_warp = -1; break; }
                  __nanosleep(64);
                }
                if (last_warp > 0) {
                  Job* jb = &jobs[items_done % kJobs];
                  jb->unit = unit;
                  jb->item0 = item0;
                  jb->nitems = nitems;
                  sts_release(&jb->seq, items_done + 1);
                }
              }
            }
            last_warp = __shfl_sync(0xffffffffu, last_warp, 0);
            if (last_warp < 0) { alive = false; break; }
            ++items_done;
          }
          break;
        }
      } else if (d.type == kSlotVB) {
        // =============================== one B item ===============================
        for (;;) {
          if (d.type != kSlotVB) { alive = false; break; }
          // ||X - v_j||^2 = ||v_j||^2 - 2 <v_j, X> + ||X||^2 for this warp's 16 tokens on the tensor
          // cores: the V rows are the A operand; used again as the B operand they give the Gram
          // blocks whose diagonals are ||v_j||^2; X, split into bf16 hi + lo columns, gives <v_j, X>.
          // Tokens for which that difference cancels (v_j close to X) or that hold most of the weight
          // are redone below by plain subtraction, so v_j = X still scores exactly 0.
          const char* sl = tiles + s * kTileBytes;
          const float* side = reinterpret_cast<const float*>(sides + s * kSideBytes);
          const FinalRec* fr = reinterpret_cast<const FinalRec*>(side + 8 * kT);
          float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f}, cx[4] = {0.f, 0.f, 0.f, 0.f};
          {
            const uint32_t vaddr = smem_u32(sl);
            const int tok = 16 * warp + 8 * (mi & 1) + mr;
            uint32_t va[8][4], xb[8][2];
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              ldmatrix_x4(vaddr + tile_off(tok, 2 * ks + (mi >> 1)), va[ks][0], va[ks][1], va[ks][2], va[ks][3]);
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              // B operand for <v, X>: column 0 = bf16 hi part of X, column 1 = lo part, the rest zero
              const float2 f0 = *reinterpret_cast<const float2*>(fr->X + 16 * ks + 2 * quad);
              const float2 f1 = *reinterpret_cast<const float2*>(fr->X + 16 * ks + 8 + 2 * quad);
              uint32_t h0, l0, h1, l1;
              split_pair(f0.x, f0.y, h0, l0);
              split_pair(f1.x, f1.y, h1, l1);
              xb[ks][0] = head == 0 ? h0 : (head == 1 ? l0 : 0u);
              xb[ks][1] = head == 0 ? h1 : (head == 1 ? l1 : 0u);
            }
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
              mma_bf16(ca, va[ks][0], va[ks][1], va[ks][2], va[ks][3], va[ks][0], va[ks][2]);  // x tokens 0..7
              mma_bf16(cb, va[ks][0], va[ks][1], va[ks][2], va[ks][3], va[ks][1], va[ks][3]);  // x tokens 8..15
              mma_bf16(cx, va[ks][0], va[ks][1], va[ks][2], va[ks][3], xb[ks][0], xb[ks][1]);
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
          const bool last = (d.flags & kFlagLast) != 0;
          release();
          if (last) break;
          if (!next_slot()) { alive = false; break; }
        }
      } else {
        alive = false;
      }
    }
    if (lane == 0) {
      if (!alive && !ctl[0]) {
        set_status(status, CAOTE_ERR_TIMEOUT);
        ctl[0] = 1;
      }
      if (warp == 0) ctl[5] = items_done;
      __threadfence_block();
      atomicAdd_block(const_cast<int*>(&ctl[4]), 1);
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
