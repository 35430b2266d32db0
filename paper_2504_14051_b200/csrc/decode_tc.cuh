// Single-query (decode) scoring path on the 5th-generation tensor cores (tcgen05 + TMEM) for bf16,
// head_dim 128, group size <= 8. Work items, records and flags: see decode_common.cuh.
//
// Every product has the tile's 128 tokens on the M side, so a token owns one TMEM lane and one thread
// from the logits to the score:
//   S^T[token][head]    = K_tile (A, K-major) x Q^T (B: 16 rows = the unit's query heads, rest unused)
//   O^T[channel][head]  = V_tile^T (A, MN-major view of the same staged bytes) x P^T (B: 16 rows =
//                         bf16 hi parts of the 8 heads' numerators, then their lo parts)
// A CTA (one per SM) runs two pipelines side by side, each fed through its own ring of shared-memory
// slots by its own producer warp (TMA):
//   attention side  K and V tiles in turn. One lane of an issuing warp queues the products; four
//                   attention warps turn S^T into softmax numerators (lazy reference: O^T is rescaled
//                   only when a logit tops the reference by more than 2^8), write the logits out and
//                   close the item (record, counter, merge by the last arriver).
//   score side      V tiles with their logits and carried base scores. Four score warps compute
//                   ||X - v_j||^2 by plain subtraction over the token's own V row, and the score.
//
// FastCAOTE (Sec. 3.3; template flag kFast): X is the plain mean of the cached values, known before
// the pass (the caller keeps the per-unit sum of V rows), so V is read once: the score warps take
// ||mean - v_j|| from the attention side's V tile while the softmax is under way and store it (4 bytes per
// token); the score side and its ring stay idle, and fast_finish_kernel turns logits, final statistics
// and distances into scores afterwards.
//
// Waits are bounded by a clock limit; the first one that runs out records CAOTE_ERR_TIMEOUT and
// raises the CTA's stop flag, after which every wait returns at once, the producers stop taking work
// and the CTA drains its copies and leaves. Indices stay in bounds whatever the buffers hold.
#pragma once

#include "decode_common.cuh"
#include "prefill_tc.cuh"

namespace caote {
namespace decode {

constexpr int kASlots = 4;                         // attention ring: K and V tiles in turn
constexpr int kBSlots = 2;                         // score ring: V tiles with their logits and base scores
constexpr int kTcTokenThreads = 128;
constexpr int kTcThreads = 2 * kTcTokenThreads + 96;  // attention warps, score warps, issuing warp, two producer warps
constexpr int kTcIssueWarp = 8, kTcProducerA = 9, kTcProducerB = 10;
constexpr int kFinBufs = 2;
constexpr int kQBytes = 2 * 16 * 128;              // 16 query rows x 128 channels, two 64-channel boxes
constexpr int kQBufs = 3;
constexpr int kPBytes = 2 * 16 * 128;              // 16 rows x 128 tokens, two 64-token boxes
constexpr uint32_t kTmemCols = 64;                 // S^T x 2 (16 columns each), O^T (16 columns)

constexpr int kBaseRowBytes = kT * 4;              // the carried base scores of one tile
constexpr int kBSideBytes = 8 * kT * 4;            // score slot: logits of up to 7 heads (rows 0..6), base scores (row 7)

constexpr int kASlotsFast = 6;                     // FastCAOTE: no score ring, a deeper attention ring instead
constexpr int kQBufsFast = 4;
constexpr int kXBufBytes = kQBufsFast * (kD + 4) * 4;  // FastCAOTE: per query buffer the sum of V rows and 1 / n

inline size_t tc_smem_bytes(bool fast) {
  const size_t a = fast ? kASlotsFast : kASlots;
  return 1024 + a * kTileBytes + (fast ? 0 : (size_t)kBSlots * kTileBytes) + (fast ? kQBufsFast : kQBufs) * kQBytes + 2 * kPBytes + a * kBaseRowBytes +
         (fast ? (size_t)kXBufBytes : (size_t)kBSlots * kBSideBytes + kFinBufs * kFinalBytes) + sizeof(Desc) * (kASlotsFast + kBSlots) +
         sizeof(float) * (2 * 4 * 8 + 4 * 8 + 4 + 8) + 8 * (2 * (kASlotsFast + kBSlots) + 8) + 64;
}

__device__ __forceinline__ void wait_or_stop(uint64_t* bar, uint32_t parity, volatile int* stop, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (*stop) return;
    if (clock64() - t0 > kWaitCycles) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      *stop = 1;
      return;
    }
  }
}
__device__ __forceinline__ void wait_or_stop_idle(uint64_t* bar, uint32_t parity, volatile int* stop, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    __nanosleep(20);
    if (*stop) return;
    if (clock64() - t0 > kWaitCycles) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      *stop = 1;
      return;
    }
  }
}
// Barrier `id` (1: attention warps, 2: score warps) of one group of token warps with an OR-reduction.
__device__ __forceinline__ bool token_any(int id, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.or.pred q, %2, %3, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred), "r"(id), "n"(kTcTokenThreads) : "memory");
  return r != 0;
}
__device__ __forceinline__ void token_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kTcTokenThreads) : "memory"); }

__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float (&v)[8]) {
  uint32_t r[8];
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])) : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}

// Two floats -> packed bf16x2 (x0 in the low half), round to nearest even.
__device__ __forceinline__ uint32_t pack_bf16x2(float x0, float x1) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x1), "f"(x0));
  return r;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 16; A K-major or MN-major, B K-major.
__host__ __device__ constexpr uint32_t idesc_n16(bool a_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
}
// k-step ks (16 of 128 contraction elements) of a 16-row K-major operand staged as two boxes of
// 16 rows x 128 bytes (128-byte swizzle): 8-row groups 1024 bytes apart, boxes 2048 bytes apart.
__device__ __forceinline__ uint64_t desc_rows16(uint32_t addr, int ks) {
  return prefill::smem_desc(addr + (ks >> 2) * 2048 + (ks & 3) * 32, 16, 1024);
}

struct Entry {  // a work item a producer is feeding into its ring
  int item, unit, item0, nitems, n, t_begin, t_end;
};

// An item's unit and tile range from the plan's item table; every lane gets the same entry.
__device__ __forceinline__ Entry find_entry(int item, const Dims& dm, const Plan& pl, const int* __restrict__ len, int lane) {
  const int4 info = __ldcg(pl.item_info + item);
  Entry e;
  e.item = item;
  e.unit = info.x;
  e.item0 = info.y;
  e.nitems = info.z;
  e.n = info.w;
  e.t_begin = (item - e.item0) * pl.tpi;
  e.t_end = min(e.t_begin + pl.tpi, (e.n + kT - 1) / kT);
  return e;
}

template <bool kFast>
__global__ void __launch_bounds__(kTcThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmQ, Dims dm, const int* __restrict__ len,
                 float* __restrict__ base, float* __restrict__ o, float* __restrict__ scores, const float* __restrict__ vsum,
                 Plan pl, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  // FastCAOTE has no score ring: its shared memory goes to a deeper attention ring
  constexpr int kA = kFast ? kASlotsFast : kASlots;
  constexpr int kQ = kFast ? kQBufsFast : kQBufs;  // a buffer is reused only after every reader of its item has moved on:
                                                   // that takes one more buffer with the deeper ring
  extern __shared__ char smem_raw[];
  // (aligned by an offset into the array, not through an integer: the pointer keeps its address space, and what is
  // read and written through it compiles to shared-memory accesses, not generic ones)
  char* sm = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  char* tilesA = sm;                                                     // [kA][kTileBytes]
  char* tilesB = tilesA + kA * kTileBytes;                               // [kBSlots][kTileBytes] (none with kFast)
  char* qbuf = tilesB + (kFast ? 0 : kBSlots * kTileBytes);                            // [kQ][kQBytes]
  char* pbuf = qbuf + kQ * kQBytes;                                  // [2][kPBytes]
  char* baseA = pbuf + 2 * kPBytes;                                      // [kA][kBaseRowBytes]
  char* sideB = baseA + kA * kBaseRowBytes;                         // [kBSlots][kBSideBytes]
  float* xbuf = reinterpret_cast<float*>(sideB);                         // kFast: [kQ][kD + 4] sum of V rows, 1 / n
  char* finbuf = sideB + (kFast ? kXBufBytes : kBSlots * kBSideBytes);                          // [kFinBufs] FinalRec
  Desc* descA = reinterpret_cast<Desc*>(finbuf + (kFast ? 0 : kFinBufs * kFinalBytes));  // [kA]
  Desc* descB = descA + kA;                                         // [kBSlots]
  float* red = reinterpret_cast<float*>(descB + kBSlots);                // [2][4][8] warp maxima
  float* wl = red + 2 * 4 * 8;                                           // [4][8] warp sums
  float* whb = wl + 4 * 8;                                               // [4]
  float* wxx = whb + 4;                                                  // [8]
  uint64_t* fullA = reinterpret_cast<uint64_t*>(wxx + 8);                // [kA]
  uint64_t* emptyA = fullA + kA;                                    // [kA] 4 attention warps + the issuing lane
  uint64_t* fullB = emptyA + kA;                                    // [kBSlots]
  uint64_t* emptyB = fullB + kBSlots;                                    // [kBSlots] 4 score warps
  uint64_t* s_bar = emptyB + kBSlots;                                    // [2] S^T formed
  uint64_t* p_bar = s_bar + 2;                                           // [2] P^T written
  uint64_t* o_bar = p_bar + 2;                                           // [2] O^T += done
  uint64_t* done_bar = o_bar + 2;                                        // [1] every product finished
  volatile int* ctl = reinterpret_cast<volatile int*>(done_bar + 2);     // [0] stop, [1] last arriver,
                                                                         // [2] / [3] slots issued in ring A / B
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(ctl) + 4);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = dm.G, mode = dm.base_mode;
  const bool use_base = (mode == CAOTE_BASE_ACCUM || mode == CAOTE_BASE_EXTERNAL);
  const bool softmax_counted = (mode != CAOTE_BASE_EXTERNAL);
  const float scale2 = dm.scale * 1.4426950408889634f;
  const int N = pl.item_prefix[dm.units];
  const int tiles_per_unit = pl.capS / kT;

  if (tid == 0) {
    for (int i = 0; i < kA; ++i) {
      mbar_init(&fullA[i], 1);
      mbar_init(&emptyA[i], kFast ? 9 : 5);  // 4 attention warps + the issuing lane (+ 4 score warps)
    }
    for (int i = 0; i < kBSlots; ++i) {
      mbar_init(&fullB[i], 1);
      mbar_init(&emptyB[i], 4);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&s_bar[i], 1);
      mbar_init(&p_bar[i], 4);
      mbar_init(&o_bar[i], 1);
    }
    mbar_init(done_bar, 1);
    ctl[0] = 0;
    ctl[1] = 0;
    ctl[2] = 0;
    ctl[3] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (tid < (kA + kBSlots) * (int)(sizeof(Desc) / sizeof(int))) reinterpret_cast<int*>(descA)[tid] = 0;
  // rows of P^T that no head writes stay zero for the whole kernel
  for (int i = tid; i < 2 * kPBytes / 16; i += kTcThreads) reinterpret_cast<uint4*>(pbuf)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  if (warp == kTcIssueWarp) prefill::tmem_alloc(tmem_slot, kTmemCols);
  prefill::tc_fence_before();
  __syncthreads();
  prefill::tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tO = tmem + 32;

  int seenA = 0, seenB = 0;  // slots whose copies these threads have seen land (thread 0 / thread 128)

  if (warp == kTcProducerA) {
    // ================================ producer of the attention ring ================================
    const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
    int issued = 0, a_items = 0, a_tiles = 0;
    bool ok = true;
    while (ok) {
      int w = 0;
      if (lane == 0) w = atomicAdd(&pl.work[0], 1);
      w = __shfl_sync(0xffffffffu, w, 0);
      if (w >= N) break;
      const Entry e = find_entry(w, dm, pl, len, lane);
      if (lane == 0) {
        for (int t = e.t_begin; ok && t < e.t_end; ++t) {
          Desc d;
          d.unit = e.unit;
          d.tile = t;
          d.n_valid = min(kT, e.n - t * kT);
          d.flags = (t == e.t_begin ? kFlagFirst : 0) | (t == e.t_end - 1 ? kFlagLast : 0);
          d.item = e.item;
          d.item0 = e.item0;
          d.nitems = e.nitems;
          const int row = e.unit * dm.cap + t * kT;
          const uint32_t base_bytes = use_base ? (uint32_t)min(kT, dm.cap - t * kT) * 4u : 0u;
          int s = issued % kA;
          if (!(ok = mbar_wait(&emptyA[s], ((issued / kA) & 1) ^ 1, &ctl[0]))) break;
          char* tl = tilesA + s * kTileBytes;
          d.type = kSlotKA;
          descA[s] = d;
          const bool first = (d.flags & kFlagFirst) != 0;
          if (kFast && first) xbuf[(a_items % kQ) * (kD + 4) + kD] = 1.f / (float)e.n;
          mbar_expect_tx(&fullA[s], kTileBytes + base_bytes + (first ? (uint32_t)kQBytes + (kFast ? kD * 4u : 0u) : 0u));
          tma_load_2d(tl, &tmK, 0, row, &fullA[s], pol_stream);
          tma_load_2d(tl + kHalfBytes, &tmK, 64, row, &fullA[s], pol_stream);
          if (use_base)
            bulk_load(baseA + (a_tiles % kA) * kBaseRowBytes, base + (size_t)e.unit * dm.cap + t * kT, base_bytes, &fullA[s]);
          ++a_tiles;
          if (first) {
            // the unit's query rows (16 rows from its first head on; only the first G are used)
            char* qb = qbuf + (a_items % kQ) * kQBytes;
            const int qrow = (e.unit / dm.Hkv) * dm.Hq + (e.unit % dm.Hkv) * G;
            tma_load_2d(qb, &tmQ, 0, qrow, &fullA[s], pol_keep);
            tma_load_2d(qb + kQBytes / 2, &tmQ, 64, qrow, &fullA[s], pol_keep);
            if (kFast) bulk_load(xbuf + (a_items % kQ) * (kD + 4), vsum + (size_t)e.unit * kD, kD * 4, &fullA[s]);
            ++a_items;
          }
          ctl[2] = ++issued;
          s = issued % kA;
          if (!(ok = mbar_wait(&emptyA[s], ((issued / kA) & 1) ^ 1, &ctl[0]))) break;
          tl = tilesA + s * kTileBytes;
          d.type = kSlotVA;
          descA[s] = d;
          mbar_expect_tx(&fullA[s], kTileBytes);
          tma_load_2d(tl, &tmV, 0, row, &fullA[s], pol_keep);
          tma_load_2d(tl + kHalfBytes, &tmV, 64, row, &fullA[s], pol_keep);
          ctl[2] = ++issued;
        }
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    if (lane == 0) {
      if (ok) {
        const int s = issued % kA;
        if (mbar_wait(&emptyA[s], ((issued / kA) & 1) ^ 1, &ctl[0])) {
          descA[s].type = kSlotStop;
          mbar_arrive(&fullA[s]);
          ctl[2] = ++issued;
        } else {
          ok = false;
        }
      }
      if (!ok && !ctl[0]) {
        set_status(status, CAOTE_ERR_TIMEOUT);
        ctl[0] = 1;
      }
    }
  } else if (warp == kTcProducerB) {
    // ================================ producer of the score ring ================================
    // Score items are taken in list order from a counter of their own; an item waits here for its
    // unit's ready flag. Attention items never wait for anything but ring slots, so every flag is
    // raised in the end, whatever the score side of any CTA is waiting for.
    const uint64_t pol_stream = policy_evict_first();
    int issued = 0, b_items = 0;
    bool ok = true;
    while (ok && !kFast) {  // (FastCAOTE has no second pass over V: this ring stays empty)
      int w = 0;
      if (lane == 0) w = atomicAdd(&pl.work[1], 1);
      w = __shfl_sync(0xffffffffu, w, 0);
      if (w >= N) break;
      const Entry e = find_entry(w, dm, pl, len, lane);
      if (lane == 0) {
        const long long t0c = clock64();
        while (ld_acquire(&pl.ready[e.unit]) == 0) {
          if (ctl[0] || clock64() - t0c > kWaitCycles) { ok = false; break; }
          __nanosleep(100);
        }
        fence_async_all();  // the record and the logits were written by other CTAs' threads
        for (int t = e.t_begin; ok && t < e.t_end; ++t) {
          Desc d;
          d.type = kSlotVB;
          d.unit = e.unit;
          d.tile = t;
          d.n_valid = min(kT, e.n - t * kT);
          d.flags = (t == e.t_begin ? kFlagFirst : 0) | (t == e.t_end - 1 ? kFlagLast : 0);
          d.item = b_items;  // which final-record buffer the item uses
          d.item0 = e.item0;
          d.nitems = e.nitems;
          const int row = e.unit * dm.cap + t * kT;
          const uint32_t base_bytes = use_base ? (uint32_t)min(kT, dm.cap - t * kT) * 4u : 0u;
          const int s = issued % kBSlots;
          if (!(ok = mbar_wait(&emptyB[s], ((issued / kBSlots) & 1) ^ 1, &ctl[0]))) break;
          char* tl = tilesB + s * kTileBytes;
          char* sd = sideB + s * kBSideBytes;
          descB[s] = d;
          const bool first = (d.flags & kFlagFirst) != 0;
          const uint32_t s_bytes = softmax_counted ? (uint32_t)G * kT * 4u : 0u;
          mbar_expect_tx(&fullB[s], kTileBytes + s_bytes + base_bytes + (first ? (uint32_t)kFinalBytes : 0u));
          tma_load_2d(tl, &tmV, 0, row, &fullB[s], pol_stream);
          tma_load_2d(tl + kHalfBytes, &tmV, 64, row, &fullB[s], pol_stream);
          if (softmax_counted)
            bulk_load(sd, pl.S + ((size_t)e.unit * tiles_per_unit + t) * G * kT, s_bytes, &fullB[s]);
          if (use_base) bulk_load(sd + 7 * kT * 4, base + (size_t)e.unit * dm.cap + t * kT, base_bytes, &fullB[s]);
          if (first) bulk_load(finbuf + (b_items % kFinBufs) * kFinalBytes, pl.fin + e.unit, kFinalBytes, &fullB[s]);
          ctl[3] = ++issued;
        }
        ++b_items;
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    if (lane == 0 && !kFast) {
      if (ok) {
        const int s = issued % kBSlots;
        if (mbar_wait(&emptyB[s], ((issued / kBSlots) & 1) ^ 1, &ctl[0])) {
          descB[s].type = kSlotStop;
          mbar_arrive(&fullB[s]);
          ctl[3] = ++issued;
        } else {
          ok = false;
        }
      }
      if (!ok && !ctl[0]) {
        set_status(status, CAOTE_ERR_TIMEOUT);
        ctl[0] = 1;
      }
    }
  } else if (warp == kTcIssueWarp) {
    // ================================ issuing warp (one lane) ================================
    if (lane == 0) {
      constexpr uint32_t kIdQK = idesc_n16(false), kIdPV = idesc_n16(true);
      int a_cnt = 0;         // attention tiles whose S^T product has been queued
      int pv_cnt = 0;        // attention tiles whose O^T product has been queued
      int q_items = 0;       // attention items whose first tile has been queued
      int qk_queued = -1;    // ring index of the last K slot whose product has been queued
      auto issue_qk = [&](int s, const Desc& d) {
        if (d.flags & kFlagFirst) ++q_items;
        const uint32_t ka = smem_u32(tilesA + s * kTileBytes);
        const uint32_t qa = smem_u32(qbuf + ((q_items - 1) % kQ) * kQBytes);
        prefill::tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          prefill::umma(tS + (a_cnt & 1) * 16, prefill::desc_k_major(ka, ks), desc_rows16(qa, ks), kIdQK, ks > 0);
        prefill::umma_commit(&s_bar[a_cnt & 1]);
        prefill::umma_commit(&emptyA[s]);  // this lane's arrival on the K slot: once the product has read it
        ++a_cnt;
      };
      for (int i = 0;; ++i) {
        if (i <= qk_queued) continue;  // a K slot whose product went out early; it may be refilled by now
        const int s = i % kA;
        wait_or_stop_idle(&fullA[s], (i / kA) & 1, &ctl[0], status);
        if (ctl[0]) break;
        const Desc d = descA[s];
        if (d.type == kSlotStop) break;
        if (d.type == kSlotKA) {
          issue_qk(s, d);
          qk_queued = i;
        } else {
          // queue the next tile's S^T first, if its K tile has landed: it then overlaps this tile's softmax
          {
            const int j = i + 1, s2 = j % kA;
            if (mbar_try_wait(&fullA[s2], (j / kA) & 1)) {
              const Desc d2 = descA[s2];
              if (d2.type == kSlotKA) {
                issue_qk(s2, d2);
                qk_queued = j;
              }
            }
          }
          wait_or_stop(&p_bar[pv_cnt & 1], (pv_cnt >> 1) & 1, &ctl[0], status);
          if (ctl[0]) break;
          prefill::tc_fence_after();
          const uint32_t va = smem_u32(tilesA + s * kTileBytes);
          const uint32_t pa = smem_u32(pbuf + (pv_cnt & 1) * kPBytes);
          const bool first = (d.flags & kFlagFirst) != 0;
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            prefill::umma(tO, prefill::desc_mn_major(va, kk), desc_rows16(pa, kk), kIdPV, !(first && kk == 0));
          prefill::umma_commit(&o_bar[pv_cnt & 1]);
          prefill::umma_commit(&emptyA[s]);  // this lane's arrival: once the product has read the V tile
          ++pv_cnt;
        }
      }
      // nothing of this CTA's may still be running in the tensor pipe when TMEM is given back
      prefill::umma_commit(done_bar);
      const int dummy = 0;
      mbar_wait(done_bar, 0, &dummy);
    }
  } else if (warp < 4) {
    // ================================ attention warps ================================
    const int tok = tid;                                   // token of the tile = TMEM lane = thread
    const uint32_t lane_base = (uint32_t)(32 * warp) << 16;
    float ref[8], lpart[8];
    float hbpart = 0.f;
#pragma unroll
    for (int g = 0; g < 8; ++g) { ref[g] = -INFINITY; lpart[g] = 0.f; }
    int a_cnt = 0, red_par = 0;

    for (;; ++seenA) {
      const int s = seenA % kA;
      const bool got = warp_mbar_wait(&fullA[s], (seenA / kA) & 1, &ctl[0], lane);
      if (token_any(1, !got)) {
        if (tid == 0 && !ctl[0]) {
          set_status(status, CAOTE_ERR_TIMEOUT);
          ctl[0] = 1;
        }
        break;
      }
      const Desc d = descA[s];
      if (d.type == kSlotStop) { ++seenA; break; }
      const int b = d.unit / dm.Hkv, h = d.unit % dm.Hkv;

      if (d.type == kSlotKA) {
        // ===================== softmax numerators of one tile =====================
        // these warps never touch the K tile itself: the slot goes back as soon as the product has read it
        __syncwarp();
        if (lane == 0) mbar_arrive(&emptyA[s]);
        const bool first = (d.flags & kFlagFirst) != 0;
        if (first) {
#pragma unroll
          for (int g = 0; g < 8; ++g) { ref[g] = -INFINITY; lpart[g] = 0.f; }
          hbpart = 0.f;
        }
        const int sb = a_cnt & 1;
        wait_or_stop(&s_bar[sb], (a_cnt >> 1) & 1, &ctl[0], status);
        prefill::tc_fence_after();
        float sv[8];
        tmem_ld8(tS + lane_base + sb * 16, sv);
        const bool valid = tok < d.n_valid;
        bool over = false;
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          sv[g] = (valid && g < G) ? sv[g] * scale2 : -INFINITY;
          over |= sv[g] > ref[g] + 8.f;
        }
        if (softmax_counted) {
          float* Sg = pl.S + ((size_t)d.unit * tiles_per_unit + d.tile) * G * kT + tok;
#pragma unroll
          for (int g = 0; g < 8; ++g)
            if (g < G) __stcg(Sg + g * kT, sv[g]);
        }
        float bval = 0.f;
        if (use_base) {
          bval = valid ? reinterpret_cast<const float*>(baseA + (a_cnt % kA) * kBaseRowBytes)[tok] : 0.f;
          hbpart += bval;
        }
        if (token_any(1, over)) {
          // a logit tops its head's reference by more than 2^8 (always on an item's first tile): move
          // the references to the maxima seen so far and rescale what has been accumulated
          float* rd = red + red_par * 32;
          red_par ^= 1;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            if (g < G) {
              float mx = sv[g];
#pragma unroll
              for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
              if (lane == 0) rd[warp * 8 + g] = mx;
            }
          }
          token_sync();
          float corr[8];
          bool changed = false;
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            corr[g] = 1.f;
            if (g < G) {
              const float nr = fmaxf(fmaxf(ref[g], fmaxf(rd[g], rd[8 + g])), fmaxf(rd[16 + g], rd[24 + g]));
              corr[g] = fast_exp2(ref[g] - nr);  // 2^-inf = 0 on an item's first tile
              changed |= nr != ref[g];
              lpart[g] *= corr[g];
              ref[g] = nr;
            }
          }
          if (!first && changed) {
            // O^T of the tiles so far (lane = channel); the previous tile's product must have finished
            const int pv = a_cnt - 1;
            wait_or_stop(&o_bar[pv & 1], (pv >> 1) & 1, &ctl[0], status);
            prefill::tc_fence_after();
            float ov[16];
            tmem_ld16(tO + lane_base, ov);
#pragma unroll
            for (int g = 0; g < 8; ++g) { ov[g] *= corr[g]; ov[8 + g] *= corr[g]; }
            tmem_st16(tO + lane_base, ov);
            prefill::tc_fence_before();
          }
        }
        // P^T rows g (hi part) and 8 + g (lo part), column = token; row 7 carries the base score
        char* pb = pbuf + sb * kPBytes + (tok >> 6) * 2048 + (tok & 7) * 2;
        const int chunk = (tok & 63) >> 3;
        float pv[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          const bool base_row = use_base && g == 7;
          pv[g] = base_row ? bval : (g < G ? fast_exp2(sv[g] - ref[g]) : 0.f);
          if (g < G) lpart[g] += pv[g];
        }
#pragma unroll
        for (int g = 0; g < 8; g += 2) {  // two heads per conversion; a row no head owns gets the zeros it holds anyway
          if (g < G || (use_base && g == 6)) {
            const uint32_t hi2 = pack_bf16x2(pv[g], pv[g + 1]);
            const uint32_t lo2 = pack_bf16x2(pv[g] - __uint_as_float(hi2 << 16), pv[g + 1] - __uint_as_float(hi2 & 0xffff0000u));
            char* at0 = pb + g * 128 + ((chunk ^ g) << 4);
            char* at1 = pb + (g + 1) * 128 + ((chunk ^ (g + 1)) << 4);
            *reinterpret_cast<unsigned short*>(at0) = (unsigned short)(hi2 & 0xffffu);
            *reinterpret_cast<unsigned short*>(at1) = (unsigned short)(hi2 >> 16);
            *reinterpret_cast<unsigned short*>(at0 + 1024) = (unsigned short)(lo2 & 0xffffu);
            *reinterpret_cast<unsigned short*>(at1 + 1024) = (unsigned short)(lo2 >> 16);
          }
        }
        if (d.n_valid < kT) {
          // rows behind the unit's length hold whatever the cache has there: clear them in the V tile
          // (next slot) so that a zero weight times a stray NaN cannot reach the accumulators
          const int s2 = (seenA + 1) % kA;
          wait_or_stop(&fullA[s2], ((seenA + 1) / kA) & 1, &ctl[0], status);
          if (!valid) {
            char* vt = tilesA + s2 * kTileBytes;
#pragma unroll
            for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4*>(vt + tile_off(tok, c)) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        fence_async_smem();
        prefill::tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&p_bar[sb]);
        ++a_cnt;
      } else if (d.type == kSlotVA) {
        // the product is queued by the issuing lane; these warps only close the item
        __syncwarp();
        if (lane == 0) mbar_arrive(&emptyA[s]);
        if (d.flags & kFlagLast) {
          const int pv = a_cnt - 1;
          wait_or_stop(&o_bar[pv & 1], (pv >> 1) & 1, &ctl[0], status);
          prefill::tc_fence_after();
          PartialRec* pr = pl.part + d.item;
          {
            float ov[16];
            tmem_ld16(tO + lane_base, ov);  // lane = channel
#pragma unroll
            for (int g = 0; g < 8; ++g) pr->o[g][tok] = ov[g] + ov[8 + g];
          }
          prefill::tc_fence_before();
#pragma unroll
          for (int g = 0; g < 8; ++g) {
            const float ls = warp_sum(lpart[g]);
            if (lane == 0) wl[warp * 8 + g] = ls;
          }
          {
            const float hs = warp_sum(hbpart);
            if (lane == 0) whb[warp] = hs;
          }
          token_sync();
#pragma unroll
          for (int g = 0; g < 8; ++g)  // (static indices keep ref[] in registers)
            if (tid == g) {
              pr->m[g] = ref[g];
              pr->l[g] = (wl[g] + wl[8 + g]) + (wl[16 + g] + wl[24 + g]);
            }
          if (tid == 8) pr->hb = use_base ? (whb[0] + whb[1]) + (whb[2] + whb[3]) : 0.f;
          token_sync();
          if (tid == 0) {
            __threadfence();
            const int old = atomicAdd(&pl.counter[d.unit], 1);
            ctl[1] = (old == d.nitems - 1);
          }
          token_sync();
          if (ctl[1]) {
            // ---------- last arriver: merge the unit's records (thread = channel) ----------
            __threadfence();
            const PartialRec* p0 = pl.part + d.item0;
            FinalRec* fr = pl.fin + d.unit;
            // two sweeps over the records, each with all of a record's loads in flight together
            float mfin[8], lfin[8], acc[8];
#pragma unroll
            for (int g = 0; g < 8; ++g) { mfin[g] = -INFINITY; lfin[g] = 0.f; acc[g] = 0.f; }
#pragma unroll 4
            for (int c = 0; c < d.nitems; ++c) {
              const float4 m0 = __ldcg(reinterpret_cast<const float4*>(p0[c].m));
              const float4 m1 = __ldcg(reinterpret_cast<const float4*>(p0[c].m + 4));
              mfin[0] = fmaxf(mfin[0], m0.x); mfin[1] = fmaxf(mfin[1], m0.y);
              mfin[2] = fmaxf(mfin[2], m0.z); mfin[3] = fmaxf(mfin[3], m0.w);
              mfin[4] = fmaxf(mfin[4], m1.x); mfin[5] = fmaxf(mfin[5], m1.y);
              mfin[6] = fmaxf(mfin[6], m1.z); mfin[7] = fmaxf(mfin[7], m1.w);
            }
            float hbsum = 0.f;
#pragma unroll 4
            for (int c = 0; c < d.nitems; ++c) {
              const float4 m0 = __ldcg(reinterpret_cast<const float4*>(p0[c].m));
              const float4 m1 = __ldcg(reinterpret_cast<const float4*>(p0[c].m + 4));
              const float4 l0 = __ldcg(reinterpret_cast<const float4*>(p0[c].l));
              const float4 l1 = __ldcg(reinterpret_cast<const float4*>(p0[c].l + 4));
              const float mc[8] = {m0.x, m0.y, m0.z, m0.w, m1.x, m1.y, m1.z, m1.w};
              const float lc[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
              hbsum += __ldcg(&p0[c].hb);
#pragma unroll
              for (int g = 0; g < 8; ++g) {
                const bool base_row = use_base && g == 7;
                if (g < G || base_row) {
                  const float f = base_row ? 1.f : exp2f(mc[g] - mfin[g]);
                  lfin[g] = fmaf(lc[g], f, lfin[g]);
                  acc[g] = fmaf(__ldcg(&p0[c].o[g][tok]), f, acc[g]);
                }
              }
            }
            const float Htot = (softmax_counted ? (float)G : 0.f) + (use_base ? hbsum : 0.f);
            float xsum = 0.f;
#pragma unroll
            for (int g = 0; g < 8; ++g) {
              const bool base_row = use_base && g == 7;
              if (base_row) {
                xsum += acc[g];
              } else if (g < G) {
                const float inv_l = 1.f / lfin[g];
                const float on = acc[g] * inv_l;
                o[((size_t)b * dm.Hq + h * G + g) * kD + tok] = on;
                if (softmax_counted) xsum += on;
                if (tid == 0) {
                  fr->m[g] = mfin[g];
                  fr->inv_l[g] = inv_l;
                  if (pl.rowstat) pl.rowstat[(size_t)d.unit * kHeadStatFloats + g] = mfin[g] + log2f(lfin[g]);
                }
              }
            }
            const float xv = (Htot > 0.f) ? xsum / Htot : 0.f;
            fr->X[tok] = xv;
            const float xx = warp_sum(xv * xv);
            if (lane == 0) wxx[warp] = xx;
            if (tid == 0) {
              fr->H = Htot;
              for (int hd = G; hd < 8; ++hd) { fr->m[hd] = 0.f; fr->inv_l[hd] = 0.f; }
            }
            token_sync();
            if (tid == 0) {
              fr->XX = (wxx[0] + wxx[1]) + (wxx[2] + wxx[3]);
              __threadfence();
              st_release(&pl.ready[d.unit], 1);
            }
          }
        }
      }
    }
  } else {
    // ================================ score warps (thread = token) ================================
    const int tok = tid - kTcTokenThreads;
    if constexpr (kFast) {
      // FastCAOTE: walk the attention ring; from every V tile take || mean(v) - v_j || of the token's row
      int items = 0;
      for (int i = 0;; ++i) {
        const int s = i % kA;
        const char* sl = tilesA + s * kTileBytes;
        const bool got = warp_mbar_wait(&fullA[s], (i / kA) & 1, &ctl[0], lane);
        if (token_any(2, !got)) {
          if (tok == 0 && !ctl[0]) {
            set_status(status, CAOTE_ERR_TIMEOUT);
            ctl[0] = 1;
          }
          break;
        }
        const Desc d = descA[s];
        if (d.type == kSlotStop) break;
        if (d.type == kSlotKA) {
          if (d.flags & kFlagFirst) ++items;
        } else {
          const float* xs = xbuf + ((items - 1) % kQ) * (kD + 4);
          const float inv_n = xs[kD];
          float n2a = 0.f, n2b = 0.f;
#pragma unroll 2
          for (int c = 0; c < 16; ++c) {
            const uint4 raw = *reinterpret_cast<const uint4*>(sl + tile_off(tok, c));
            const float4 x0 = *reinterpret_cast<const float4*>(xs + 8 * c);
            const float4 x1 = *reinterpret_cast<const float4*>(xs + 8 * c + 4);
            const float d0 = fmaf(x0.x, inv_n, -__uint_as_float(raw.x << 16)), d1 = fmaf(x0.y, inv_n, -__uint_as_float(raw.x & 0xffff0000u));
            const float d2 = fmaf(x0.z, inv_n, -__uint_as_float(raw.y << 16)), d3 = fmaf(x0.w, inv_n, -__uint_as_float(raw.y & 0xffff0000u));
            const float d4 = fmaf(x1.x, inv_n, -__uint_as_float(raw.z << 16)), d5 = fmaf(x1.y, inv_n, -__uint_as_float(raw.z & 0xffff0000u));
            const float d6 = fmaf(x1.z, inv_n, -__uint_as_float(raw.w << 16)), d7 = fmaf(x1.w, inv_n, -__uint_as_float(raw.w & 0xffff0000u));
            n2a = fmaf(d0, d0, n2a); n2b = fmaf(d1, d1, n2b);
            n2a = fmaf(d2, d2, n2a); n2b = fmaf(d3, d3, n2b);
            n2a = fmaf(d4, d4, n2a); n2b = fmaf(d5, d5, n2b);
            n2a = fmaf(d6, d6, n2a); n2b = fmaf(d7, d7, n2b);
          }
          if (tok < d.n_valid) __stcg(pl.dist + (size_t)d.unit * pl.capS + (size_t)d.tile * kT + tok, sqrtf(n2a + n2b));
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&emptyA[s]);
      }
    } else
    for (;; ++seenB) {
      const int s = seenB % kBSlots;
      const char* sl = tilesB + s * kTileBytes;
      const float* side = reinterpret_cast<const float*>(sideB + s * kBSideBytes);
      const bool got = warp_mbar_wait(&fullB[s], (seenB / kBSlots) & 1, &ctl[0], lane);
      if (token_any(2, !got)) {
        if (tok == 0 && !ctl[0]) {
          set_status(status, CAOTE_ERR_TIMEOUT);
          ctl[0] = 1;
        }
        break;
      }
      const Desc d = descB[s];
      if (d.type == kSlotStop) { ++seenB; break; }
      const FinalRec* fr = reinterpret_cast<const FinalRec*>(finbuf + (d.item % kFinBufs) * kFinalBytes);
      const bool valid = tok < d.n_valid;
      float hj = 0.f;
      if (softmax_counted) {
#pragma unroll
        for (int g = 0; g < 8; ++g)
          if (g < G) hj = fmaf(fast_exp2(side[g * kT + tok] - fr->m[g]), fr->inv_l[g], hj);
      }
      const size_t slot = (size_t)d.unit * dm.cap + (size_t)d.tile * kT + tok;
      if (valid) {
        if (mode == CAOTE_BASE_ACCUM) {
          hj += side[7 * kT + tok];
          base[slot] = hj;
        } else if (mode == CAOTE_BASE_EXTERNAL) {
          hj = side[7 * kT + tok];
        }
      }
      float n2a = 0.f, n2b = 0.f;
#pragma unroll 2
      for (int c = 0; c < 16; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(sl + tile_off(tok, c));
        const float4 x0 = *reinterpret_cast<const float4*>(fr->X + 8 * c);
        const float4 x1 = *reinterpret_cast<const float4*>(fr->X + 8 * c + 4);
        const float d0 = x0.x - __uint_as_float(raw.x << 16), d1 = x0.y - __uint_as_float(raw.x & 0xffff0000u);
        const float d2 = x0.z - __uint_as_float(raw.y << 16), d3 = x0.w - __uint_as_float(raw.y & 0xffff0000u);
        const float d4 = x1.x - __uint_as_float(raw.z << 16), d5 = x1.y - __uint_as_float(raw.z & 0xffff0000u);
        const float d6 = x1.z - __uint_as_float(raw.w << 16), d7 = x1.w - __uint_as_float(raw.w & 0xffff0000u);
        n2a = fmaf(d0, d0, n2a); n2b = fmaf(d1, d1, n2b);
        n2a = fmaf(d2, d2, n2a); n2b = fmaf(d3, d3, n2b);
        n2a = fmaf(d4, d4, n2a); n2b = fmaf(d5, d5, n2b);
        n2a = fmaf(d6, d6, n2a); n2b = fmaf(d7, d7, n2b);
      }
      if (valid) {
        const float Htot = fr->H;
        float ratio = 0.f;
        if (Htot > 0.f) {
          const float rest = Htot - hj;
          ratio = (rest > 0.f) ? hj / rest : INFINITY;
        }
        scores[slot] = (ratio == 0.f) ? 0.f : ((ratio == INFINITY) ? INFINITY : ratio * sqrtf(n2a + n2b));
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&emptyB[s]);
    }
  }

  // Leave only after every copy this CTA issued has landed (bounded), whatever the reason for leaving.
  prefill::tc_fence_before();
  __syncthreads();
  prefill::tc_fence_after();
  const int dummy = 0;
  if (tid == 0)
    for (int j = seenA; j < ctl[2]; ++j) mbar_wait(&fullA[j % kA], (j / kA) & 1, &dummy);
  if (tid == kTcTokenThreads)
    for (int j = seenB; j < ctl[3]; ++j) mbar_wait(&fullB[j % kBSlots], (j / kBSlots) & 1, &dummy);
  if (warp == kTcIssueWarp) prefill::tmem_dealloc(tmem, kTmemCols);
}

// FastCAOTE, after decode_tc_kernel<true>: c_j = w_j / (1 - w_j) * || mean(v) - v_j || from the stored
// logits, the unit's final softmax statistics and the stored distances. grid = (tiles, units), kT threads.
__global__ void __launch_bounds__(kT)
fast_finish_kernel(Dims dm, const int* __restrict__ len, float* __restrict__ base, float* __restrict__ scores, Plan pl) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  const int unit = blockIdx.y, tile = blockIdx.x, b = unit / dm.Hkv;
  const int n = len[b], tok = tile * kT + threadIdx.x;
  if (n <= 0 || n > dm.cap || tok >= n) return;
  const int G = dm.G, mode = dm.base_mode;
  const FinalRec* fr = pl.fin + unit;
  float hj = 0.f;
  if (mode != CAOTE_BASE_EXTERNAL) {
    const float* Sg = pl.S + ((size_t)unit * (pl.capS / kT) + tile) * G * kT + threadIdx.x;
    for (int g = 0; g < G; ++g) hj = fmaf(fast_exp2(__ldcg(Sg + g * kT) - fr->m[g]), fr->inv_l[g], hj);
  }
  const size_t slot = (size_t)unit * dm.cap + tok;
  if (mode == CAOTE_BASE_ACCUM) {
    hj += base[slot];
    base[slot] = hj;
  } else if (mode == CAOTE_BASE_EXTERNAL) {
    hj = base[slot];
  }
  const float Htot = fr->H;
  float ratio = 0.f;
  if (Htot > 0.f) {
    const float rest = Htot - hj;
    ratio = (rest > 0.f) ? hj / rest : INFINITY;
  }
  const float dist = __ldcg(pl.dist + (size_t)unit * pl.capS + tok);
  scores[slot] = (ratio == 0.f) ? 0.f : ((ratio == INFINITY) ? INFINITY : ratio * dist);
}

}  // namespace decode
}  // namespace caote
