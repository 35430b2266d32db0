// Single-query (decode) scoring path, bf16, head_dim 128, group size <= 8: one thread-block cluster per
// (sequence, KV head) unit, K and V read from HBM exactly once.
//
// Why a cluster. The score c_j = w_j / (1 - w_j) * ||X - v_j|| needs every value row twice: once for
// the attention output (which gives X) and once more, after X is known, for the distance. A unit's
// cluster keeps the value rows on chip between the two uses, so the second use costs no HBM traffic:
//   * the unit's 128-token tiles are dealt to the C CTAs of the cluster (at most kMaxT each);
//   * attention pass: K and V tiles stream through two TMA rings; S^T = K_tile Q^T and
//     O^T += V_tile^T P^T run on tcgen05 with the tile's tokens on the M side (a token owns one TMEM
//     lane); the softmax group turns S^T into P^T; the keeper group copies every token's value row (256
//     bytes) from the landed V tile into a TMEM stash slot (64 columns per tile, 7 slots beside the
//     accumulators; a CTA's tiles beyond the 7th stay in their V ring slot instead) and keeps the
//     token's logits in registers;
//   * merge: the softmax group pushes its (reference, sums, partial output) record to the peers through
//     distributed shared memory (st.async, completion counted by an mbarrier of the receiver): the
//     softmax statistics go to everyone, the partial outputs to the CTA that owns the channel slice;
//     the keeper groups finish o and X for their channels and push X to everyone;
//   * score pass: the keeper group takes its tokens' rows back from the stash, forms ||X - v_j||^2 by
//     plain subtraction and writes c_j -- while the softmax group is already busy with the next unit.
// Nothing but q, K, V, base are read from global memory and nothing but o, scores, base is written.
//
// 1 - w_j without cancellation (Sec. 3.2 normalisation; a token that holds almost all the weight): per
// head the largest numerator is kept apart from the sum of the others, through the thread, the warp,
// the CTA and the cluster, so that the complement of the head's top token is l_rest / l (a sum of the
// other tokens' numerators) and every other token's complement is 1 - alpha with alpha <= 1/2; the
// carried base scores are treated the same way. The heads' complements, all non-negative, are added.
//
// Warp roles (512 threads): warps 0..3 softmax group, then kNB = 2 keeper groups of four warps that take the
// CTA's tiles in turn (thread = token = TMEM lane in all of them); one lane each of the last four warps
// issues the K copies, the V copies, the S^T products and the O^T products. Several token warps per
// scheduler: a single warp cannot hide the latency of its own instruction stream. (Three keeper groups at
// 96 registers per thread were slower: 246 us against 218 us on the batched 8k-token decode workload.)
//
// Flow control between units. Buffers that peers write (records, X) are reused every unit. A record of
// unit u + 1 is pushed only after this CTA has seen round 2 of unit u complete, and round 2 includes a
// word from every peer sent after that peer has finished reading its copies of unit u's records; X is
// double-buffered by unit parity. So no push can overtake a read, and no mbarrier phase can receive
// bytes of the next one.
//
// Every wait is bounded by a clock limit. A wait that runs out records CAOTE_ERR_TIMEOUT and raises the
// CTA's stop flag; from then on no wait of this CTA blocks, the copy and product issuers stop, the token
// groups run through the rest of their schedule on whatever their buffers hold (indices stay in bounds,
// results are meaningless and the status word says so), and the CTA still drains its copies, frees its
// TMEM and meets its peers at the closing cluster barrier, so that nobody writes into the shared memory
// of a CTA that has left.
#pragma once

#include "decode_tc.cuh"

namespace caote {
namespace dcl {

using decode::bulk_load;
using decode::fast_exp2;
using decode::fence_async_smem;
using decode::idesc_n16;
using decode::kD;
using decode::kHalfBytes;
using decode::kT;
using decode::kTileBytes;
using decode::mbar_arrive;
using decode::mbar_expect_tx;
using decode::mbar_init;
using decode::mbar_try_wait;
using decode::pack_bf16x2;
using decode::smem_u32;
using decode::tile_off;
using decode::tma_load_2d;
using decode::tmem_ld16;
using decode::tmem_ld8;
using decode::tmem_st16;

constexpr int kKS = 2;                    // K ring slots (a slot is free as soon as S^T is formed)
constexpr int kVS = 4;                    // V ring slots (free after O^T += and the stash copy)
constexpr int kSB = 3;                    // S^T buffers in TMEM (free once both groups have read them)
constexpr int kStash = 7;                 // value tiles a CTA keeps in TMEM
constexpr int kMaxT = 9;                  // tiles of one unit per CTA: the stash + 2 held in the V ring
constexpr int kMaxC = 16;                 // largest cluster
constexpr int kGroup = 128;               // threads of a token group
constexpr int kNB = 2;                    // keeper groups
constexpr int kThreads = (1 + kNB) * kGroup + 128;  // softmax group, keeper groups, four single-lane warps
constexpr int kWarpK = 4 * (1 + kNB), kWarpV = kWarpK + 1, kWarpQK = kWarpK + 2, kWarpPV = kWarpK + 3;
constexpr int kMaxKeep = (kMaxT + kNB - 1) / kNB;   // tiles of one unit per keeper group
constexpr int kQBufBytes = 2048;          // 8 query rows x 128 channels as two 64-channel boxes
constexpr int kPBytes = 4096;             // 16 rows x 128 tokens as two 64-token boxes
constexpr int kStatFloats = 36;           // per CTA: ref[8] lrest[8] pmax[8] smax[8] brest bmax pad pad
constexpr int kXoFloats = 8 * (kD + kMaxC);  // partial outputs received: [C][slice][8], slice = ceil(128 / C)
constexpr int kLenTab = 512;              // unit lengths of this cluster kept in shared memory
constexpr uint32_t kTmemCols = 512;       // S^T x 3, O^T (16 columns each), 7 stash slots of 64 columns
constexpr long long kDrainCycles = 4000000000LL;  // waits for hardware to finish what was already issued

struct Fin {        // per unit, every CTA computes its own copy
  float m[8];       // final softmax reference per head (log2 domain) + log2 of the sum of numerators:
                    // alpha_j = 2^(s_j - m)
  float inv_l[8];   // 1 / sum_j 2^(s_j - reference)
  float smax[8];    // largest logit of the head
  float crest[8];   // (sum of the numerators of all tokens but the head's top one) / l
  float Htot;       // normaliser of the base score
  float hbsum;      // sum of the carried base scores
  float bmax;       // largest carried base score
  float brest;      // sum of the other carried base scores
};

inline size_t smem_bytes() {
  return 1024 + (size_t)(kKS + kVS) * kTileBytes + 2 * kQBufBytes + kPBytes + kVS * (kT * 4) +
         kMaxC * kStatFloats * 4 + kXoFloats * 4 + 2 * kD * 4 + kNB * sizeof(Fin) + kNB * kMaxC * 8 * 4 /* fac */ +
         2 * 32 * 4 /* red */ + 4 * 28 * 4 /* gred */ + kStatFloats * 4 /* mystat */ + kLenTab * 4 + 64 * 8 /* barriers, control words */ + 64;
}

// ---- cluster PTX (the register reads, mapa and the cluster barrier are in ptx.cuh) ----------------------
using ptx::cluster_count_x;
using ptx::cluster_ctarank;
using ptx::cluster_id_x;
using ptx::cluster_nctarank;
using ptx::cluster_sync_all;
using ptx::map_to_rank;
// Floats into a peer's shared memory; the peer's mbarrier counts the bytes when they have landed.
__device__ __forceinline__ void push_f32(uint32_t remote_addr, float v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(remote_addr), "r"(__float_as_uint(v)), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void push_f32x4(uint32_t remote_addr, float a, float b, float c, float d, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(remote_addr), "r"(__float_as_uint(a)), "r"(__float_as_uint(b)), "r"(__float_as_uint(c)),
                 "r"(__float_as_uint(d)), "r"(remote_bar) : "memory");
}

// try_wait that lets the hardware park the thread until the phase completes or `ns` nanoseconds pass: a
// waiting warp then takes no issue slots and no shared-memory bandwidth from the warps that work.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(ns) : "memory");
  return ok != 0;
}

// Wait for hardware to finish what has already been issued (copies in flight, queued products).
__device__ __noinline__ void drain_wait(uint64_t* bar, uint32_t parity, int* status) {
  const long long t0 = clock64();
  while (!mbar_try_wait_parked(bar, parity, 2000u)) {
    if (clock64() - t0 > kDrainCycles) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      return;
    }
  }
}
// Bounded wait; a wait that runs out records the timeout and raises the stop flag. Never blocks once the
// flag is up. The polling loop is kept out of line: the common case is that the phase has completed.
__device__ __noinline__ void wait_slow(uint64_t* bar, uint32_t parity, volatile int* stop, int* status, long long limit,
                                       bool idle) {
  const long long t0 = clock64();
  while (!mbar_try_wait_parked(bar, parity, 2000u)) {
    if (*stop) return;
    if (clock64() - t0 > limit) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      *stop = 1;
      return;
    }
  }
}
__device__ __forceinline__ void wait_bounded(uint64_t* bar, uint32_t parity, volatile int* stop, int* status,
                                             long long limit, bool idle) {
  if (mbar_try_wait(bar, parity) || *stop) return;
  wait_slow(bar, parity, stop, status, limit, idle);
}
// Barrier of one token group (id 1: softmax group, id 2: keeper group), with and without an OR-reduction.
__device__ __forceinline__ bool group_any(int g, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 p, %1, 0;\n\t"
      "bar.red.or.pred q, %2, %3, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r) : "r"((uint32_t)pred), "r"(1 + g), "n"(kGroup) : "memory");
  return r != 0;
}
__device__ __forceinline__ void group_sync(int g) { asm volatile("bar.sync %0, %1;" ::"r"(1 + g), "n"(kGroup) : "memory"); }

__device__ __forceinline__ void tmem_ld16u(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// sqrt, hardware approximation (about 1 ulp).
__device__ __forceinline__ float fast_sqrt(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// k-step ks of the query operand: two boxes of 8 rows x 128 bytes, 1024 bytes apart. The product reads 16
// rows (N = 16); rows 8..15 fall on whatever follows in shared memory and only feed unused columns.
__device__ __forceinline__ uint64_t desc_q(uint32_t addr, int ks) {
  return prefill::smem_desc(addr + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 1024);
}

// (sum of the others, largest, its logit) of two disjoint sets of tokens -> of their union.
__device__ __forceinline__ void top_merge(float& l, float& p, float& s, float ol, float op, float os) {
  const bool mine = s >= os;
  l = l + ol + (mine ? op : p);
  p = mine ? p : op;
  s = fmaxf(s, os);
}

// ---- the static schedule ------------------------------------------------------------------------------
// The k-th unit of cluster `cid` is unit cid + k * ncl. Its nt tiles are dealt to the C ranks in contiguous
// runs of floor(nt / C) or that plus one; which ranks get the longer runs rotates with k.
struct Work {
  int unit, n, t0, T;
  bool ok;  // 0 < n <= cap
};
struct Sched {
  int C, rank, cid, ncl, units, Hkv, cap;
  const int* len;
  const int* slen;  // the first kLenTab lengths of this cluster's units (shared memory)
  __device__ __forceinline__ int count() const { return cid < units ? (units - cid + ncl - 1) / ncl : 0; }
  __device__ __forceinline__ Work at(int k) const {
    Work w;
    w.unit = cid + k * ncl;
    w.n = (k < kLenTab) ? slen[k] : __ldg(len + w.unit / Hkv);
    w.ok = w.n > 0 && w.n <= cap;
    const int nt = w.ok ? (w.n + kT - 1) / kT : 0;
    const int base = nt / C, rem = nt % C;
    const int rr = (rank + k) % C;
    w.T = base + (rr < rem ? 1 : 0);
    w.t0 = rr * base + min(rr, rem);
    return w;
  }
};

// kG: query heads per KV head; kMode: the base mode. Compile-time so that the per-head loops carry no
// predicates and the paths of the other modes are not in the instruction stream.
template <int kG, int kMode>
__global__ void __launch_bounds__(kThreads, 1)
decode_cluster_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                      const __grid_constant__ CUtensorMap tmQ, Dims dm, const int* __restrict__ len,
                      float* __restrict__ base, float* __restrict__ o, float* __restrict__ scores, int* status,
                      long long wait_cycles, const float* __restrict__ vsum) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  extern __shared__ char smem_raw[];
  // (aligned by an offset into the array, not through an integer: the pointer keeps its address space, and what is
  // read and written through it compiles to shared-memory accesses, not generic ones)
  char* sm = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  char* tilesK = sm;                                                   // [kKS][kTileBytes]
  char* tilesV = tilesK + kKS * kTileBytes;                            // [kVS][kTileBytes]
  char* qbuf = tilesV + kVS * kTileBytes;                              // [2][kQBufBytes]
  char* pbuf = qbuf + 2 * kQBufBytes;                                  // [kPBytes]
  float* baseV = reinterpret_cast<float*>(pbuf + kPBytes);             // [kVS][kT] carried base scores of a V slot's tile
  float* xstats = baseV + kVS * kT;                                    // [C][kStatFloats]    written by the peers
  float* xo = xstats + kMaxC * kStatFloats;                            // [C][slice][8]       written by the peers
  float* xnX = xo + kXoFloats;                                         // [2][kD]  -X         written by the owners
  Fin* fins = reinterpret_cast<Fin*>(xnX + 2 * kD);                    // [kNB] one copy per keeper group
  float* facs = reinterpret_cast<float*>(fins + kNB);                  // [kNB][C][8] 2^(ref_c - m) / l per record and head
  float* red = facs + kNB * kMaxC * 8;                                       // [2][4][8] warp maxima of the softmax group
  float* gred = red + 2 * 32;                                          // [4 warps][28] closing sums of the softmax group
  float* mystat = gred + 4 * 28;                                       // [kStatFloats] this CTA's record
  int* slen = reinterpret_cast<int*>(mystat + kStatFloats);            // [kLenTab]
  uint64_t* bars = reinterpret_cast<uint64_t*>(slen + kLenTab);
  uint64_t* kfull = bars;                 // [kKS]
  uint64_t* kempty = kfull + kKS;         // [kKS]   the S^T product has read the slot
  uint64_t* vfull = kempty + kKS;         // [kVS]
  uint64_t* vempty = vfull + kVS;         // [kVS]   4 keeper warps + the O^T product
  uint64_t* sfull = vempty + kVS;         // [kSB]   S^T of a tile is formed
  uint64_t* sfree = sfull + kSB;          // [kSB]   both groups have read it (8 warps)
  uint64_t* pfull = sfree + kSB;          // P^T of a tile is written (4 warps)
  uint64_t* odone = pfull + 1;            // O^T += of a tile is done
  uint64_t* qfree = odone + 1;            // [2]     the last S^T product of the unit that used the buffer is done
  uint64_t* r1 = qfree + 2;               // the records of all CTAs have landed
  uint64_t* r2 = r1 + 1;                  // X has landed and every peer is done with its copies of the records
  uint64_t* done_bar = r2 + 1;            // [2]     every product of an issuer has finished
  volatile int* ctl = reinterpret_cast<volatile int*>(done_bar + 2);   // [0] stop, [1] K copies issued, [2] V copies issued
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(ctl) + 4);
  float* xword = reinterpret_cast<float*>(tmem_slot + 1);              // where the peers' "done reading" words land

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int G = kG, mode = kMode;
  constexpr bool use_base = (mode == CAOTE_BASE_ACCUM || mode == CAOTE_BASE_EXTERNAL);
  constexpr bool counted = (mode != CAOTE_BASE_EXTERNAL);
  const float scale2 = dm.scale * 1.4426950408889634f;

  Sched sch;
  sch.C = (int)cluster_nctarank();
  sch.rank = (int)cluster_ctarank();
  sch.cid = (int)cluster_id_x();
  sch.ncl = (int)cluster_count_x();
  sch.units = dm.units;
  sch.Hkv = dm.Hkv;
  sch.cap = dm.cap;
  sch.len = len;
  sch.slen = slen;
  const int C = sch.C, rank = sch.rank;
  const int nk = sch.count();
  const int slice = (kD + C - 1) / C;                                   // channels per owner
  const int my_ch0 = min(rank * slice, kD), my_nch = min(slice, kD - my_ch0);
  const uint32_t r1_bytes = (uint32_t)(C * (kStatFloats * 4 + 8 * my_nch * 4));
  const uint32_t r2_bytes = (uint32_t)(kD * 4 + kNB * C * 4);

  if (tid == 0) {
    for (int i = 0; i < kKS; ++i) { mbar_init(&kfull[i], 1); mbar_init(&kempty[i], 1); }
    for (int i = 0; i < kVS; ++i) { mbar_init(&vfull[i], 1); mbar_init(&vempty[i], 5); }  // 4 keeper warps + the product
    for (int i = 0; i < kSB; ++i) { mbar_init(&sfull[i], 1); mbar_init(&sfree[i], 8); }
    mbar_init(pfull, 4);
    mbar_init(odone, 1);
    for (int i = 0; i < 2; ++i) { mbar_init(&qfree[i], 1); mbar_init(&done_bar[i], 1); }
    mbar_init(r1, 1);
    mbar_init(r2, 1);
    ctl[0] = 0;
    ctl[1] = 0;
    ctl[2] = 0;
    if (blockIdx.x == 0) status[kStatTagIndex] = kStatPerHead;  // which statistics this call leaves behind
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // the first unit's merge: what the peers will push into this CTA
    mbar_expect_tx(r1, r1_bytes);
    mbar_expect_tx(r2, r2_bytes);
  }
  for (int k = tid; k < min(nk, kLenTab); k += kThreads) slen[k] = __ldg(len + (sch.cid + k * sch.ncl) / dm.Hkv);
  // rows of P^T that no head writes stay zero for the whole kernel
  for (int i = tid; i < kPBytes / 16; i += kThreads) reinterpret_cast<uint4*>(pbuf)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  if (warp == kWarpQK) prefill::tmem_alloc(tmem_slot, kTmemCols);
  prefill::tc_fence_before();
  __syncthreads();
  prefill::tc_fence_after();
  cluster_sync_all();  // every peer's barriers exist before anyone pushes to them
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tO = tmem + 48, tStash = tmem + 64;

  if (warp == kWarpK) {
    // ================================ K copies (one lane) ================================
    if (lane == 0) {
      const uint64_t pol = decode::policy_evict_first();
      int ki = 0, us = 0;
      for (int k = 0; k < nk && !ctl[0]; ++k) {
        const Work w = sch.at(k);
        if (!w.ok || w.T == 0) continue;
        const int b = w.unit / dm.Hkv, h = w.unit % dm.Hkv;
        for (int j = 0; j < w.T; ++j) {
          const int s = ki % kKS;
          wait_bounded(&kempty[s], ((ki / kKS) & 1) ^ 1, &ctl[0], status, wait_cycles, true);
          if (j == 0) wait_bounded(&qfree[us & 1], ((us >> 1) & 1) ^ 1, &ctl[0], status, wait_cycles, true);
          if (ctl[0]) break;
          const int row = w.unit * dm.cap + (w.t0 + j) * kT;
          char* tl = tilesK + s * kTileBytes;
          mbar_expect_tx(&kfull[s], kTileBytes + (j == 0 ? (uint32_t)kQBufBytes : 0u));
          tma_load_2d(tl, &tmK, 0, row, &kfull[s], pol);
          tma_load_2d(tl + kHalfBytes, &tmK, 64, row, &kfull[s], pol);
          if (j == 0) {
            char* qb = qbuf + (us & 1) * kQBufBytes;
            const int qrow = b * dm.Hq + h * G;
            tma_load_2d(qb, &tmQ, 0, qrow, &kfull[s], pol);
            tma_load_2d(qb + kQBufBytes / 2, &tmQ, 64, qrow, &kfull[s], pol);
          }
          ctl[1] = ++ki;
        }
        ++us;
      }
    }
  } else if (warp == kWarpV) {
    // ================================ V copies (one lane) ================================
    if (lane == 0) {
      const uint64_t pol = decode::policy_evict_first();
      int vi = 0;
      for (int k = 0; k < nk && !ctl[0]; ++k) {
        const Work w = sch.at(k);
        if (!w.ok) continue;
        for (int j = 0; j < w.T; ++j) {
          const int s = vi % kVS;
          wait_bounded(&vempty[s], ((vi / kVS) & 1) ^ 1, &ctl[0], status, wait_cycles, true);
          if (ctl[0]) break;
          const int t = w.t0 + j;
          const int row = w.unit * dm.cap + t * kT;
          const uint32_t base_bytes = use_base ? (uint32_t)min(kT, dm.cap - t * kT) * 4u : 0u;
          char* tl = tilesV + s * kTileBytes;
          mbar_expect_tx(&vfull[s], kTileBytes + base_bytes);
          tma_load_2d(tl, &tmV, 0, row, &vfull[s], pol);
          tma_load_2d(tl + kHalfBytes, &tmV, 64, row, &vfull[s], pol);
          if (use_base) bulk_load(baseV + s * kT, base + (size_t)w.unit * dm.cap + (size_t)t * kT, base_bytes, &vfull[s]);
          ctl[2] = ++vi;
        }
      }
    }
  } else if (warp == kWarpQK) {
    // ================================ S^T products (one lane) ================================
    if (lane == 0) {
      constexpr uint32_t kIdQK = idesc_n16(false);
      int ki = 0, us = 0;
      for (int k = 0; k < nk && !ctl[0]; ++k) {
        const Work w = sch.at(k);
        if (!w.ok || w.T == 0) continue;
        const uint32_t qa = smem_u32(qbuf + (us & 1) * kQBufBytes);
        for (int j = 0; j < w.T; ++j) {
          const int s = ki % kKS, sb = ki % kSB;
          wait_bounded(&kfull[s], (ki / kKS) & 1, &ctl[0], status, wait_cycles, true);
          wait_bounded(&sfree[sb], ((ki / kSB) & 1) ^ 1, &ctl[0], status, wait_cycles, true);
          if (ctl[0]) break;
          prefill::tc_fence_after();
          const uint32_t ka = smem_u32(tilesK + s * kTileBytes);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            prefill::umma(tS + sb * 16, prefill::desc_k_major(ka, ks), desc_q(qa, ks), kIdQK, ks > 0);
          prefill::umma_commit(&sfull[sb]);
          prefill::umma_commit(&kempty[s]);
          if (j == w.T - 1) prefill::umma_commit(&qfree[us & 1]);
          ++ki;
        }
        ++us;
      }
      // nothing of this CTA's may still be running in the tensor pipe when TMEM is given back
      prefill::umma_commit(&done_bar[0]);
      if (!mbar_try_wait(&done_bar[0], 0)) drain_wait(&done_bar[0], 0, status);
    }
  } else if (warp == kWarpPV) {
    // ================================ O^T products (one lane) ================================
    if (lane == 0) {
      constexpr uint32_t kIdPV = idesc_n16(true);
      const uint32_t pa = smem_u32(pbuf);
      int vi = 0;
      for (int k = 0; k < nk && !ctl[0]; ++k) {
        const Work w = sch.at(k);
        if (!w.ok) continue;
        for (int j = 0; j < w.T; ++j) {
          const int s = vi % kVS;
          wait_bounded(&vfull[s], (vi / kVS) & 1, &ctl[0], status, wait_cycles, true);
          wait_bounded(pfull, vi & 1, &ctl[0], status, wait_cycles, false);
          if (ctl[0]) break;
          prefill::tc_fence_after();
          const uint32_t va = smem_u32(tilesV + s * kTileBytes);
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)  // the unit's first tile starts a new sum
            prefill::umma(tO, prefill::desc_mn_major(va, kk), decode::desc_rows16(pa, kk), kIdPV, !(j == 0 && kk == 0));
          prefill::umma_commit(odone);
          prefill::umma_commit(&vempty[s]);
          ++vi;
        }
      }
      prefill::umma_commit(&done_bar[1]);
      if (!mbar_try_wait(&done_bar[1], 0)) drain_wait(&done_bar[1], 0, status);
    }
  } else if (warp < 4) {
    // ================================ softmax group (thread = token of the tile) ================================
    const int gw = warp;
    const int tok = tid;
    const uint32_t lane_base = (uint32_t)(32 * gw) << 16;
    char* pb_tok = pbuf + (tok >> 6) * 2048 + (tok & 7) * 2;
    const int pchunk = (tok & 63) >> 3;
    int ti = 0;       // tiles this CTA has been through (phases of sfull / pfull / odone, V ring position)
    int mu = 0;       // units merged so far (phase of r2)
    int red_par = 0;

    for (int k = 0; k < nk; ++k) {
      const Work w = sch.at(k);
      if (!w.ok) {
        if (w.n != 0 && tid == 0 && rank == 0) set_status(status, CAOTE_ERR_BAD_LENGTH);
        continue;
      }
      float ref[8], lrest[8], pmax[8], smax[8];
      float brest = 0.f, bmax = 0.f;
#pragma unroll
      for (int hd = 0; hd < 8; ++hd) { ref[hd] = -INFINITY; lrest[hd] = 0.f; pmax[hd] = 0.f; smax[hd] = -INFINITY; }

#pragma unroll 1
      for (int j = 0; j < w.T; ++j, ++ti) {
        const int t = w.t0 + j;
        const int n_valid = min(kT, w.n - t * kT);
        const int vs = ti % kVS, sb = ti % kSB;
        const uint32_t vpar = (ti / kVS) & 1;
        wait_bounded(&sfull[sb], (ti / kSB) & 1, &ctl[0], status, wait_cycles, false);
        prefill::tc_fence_after();
        float sv[8];
        tmem_ld8(tS + lane_base + sb * 16, sv);
        prefill::tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sfree[sb]);
        const bool valid = tok < n_valid;
        bool over = false;
#pragma unroll
        for (int hd = 0; hd < 8; ++hd) {
          sv[hd] = (valid && hd < G) ? sv[hd] * scale2 : -INFINITY;
          over |= sv[hd] > ref[hd] + 8.f;
        }
        if (group_any(0, over)) {
          // a logit tops its head's reference by more than 2^8 (always on the unit's first tile): move
          // the references to the maxima seen so far and rescale what has been accumulated
          float* rd = red + red_par * 32;
          red_par ^= 1;
#pragma unroll
          for (int hd = 0; hd < 8; ++hd) {
            if (hd < G) {
              const float mx = warp_max(sv[hd]);
              if (lane == 0) rd[gw * 8 + hd] = mx;
            }
          }
          group_sync(0);
          float corr[8];
          bool changed = false;
#pragma unroll
          for (int hd = 0; hd < 8; ++hd) {
            corr[hd] = 1.f;
            if (hd < G) {
              const float nr = fmaxf(fmaxf(ref[hd], fmaxf(rd[hd], rd[8 + hd])), fmaxf(rd[16 + hd], rd[24 + hd]));
              corr[hd] = fast_exp2(ref[hd] - nr);  // 2^-inf = 0 on the unit's first tile
              changed |= nr != ref[hd];
              lrest[hd] *= corr[hd];
              pmax[hd] *= corr[hd];
              ref[hd] = nr;
            }
          }
          if (j > 0 && changed) {
            // O^T of the tiles so far (lane = channel); the previous product must have finished
            wait_bounded(odone, (ti - 1) & 1, &ctl[0], status, wait_cycles, false);
            prefill::tc_fence_after();
            float ov[16];
            tmem_ld16(tO + lane_base, ov);
#pragma unroll
            for (int hd = 0; hd < 8; ++hd) { ov[hd] *= corr[hd]; ov[8 + hd] *= corr[hd]; }
            tmem_st16(tO + lane_base, ov);
            prefill::tc_fence_before();
          }
        }
        // numerators; per head the largest one so far is kept apart from the sum of the others
        float pv[8];
#pragma unroll
        for (int hd = 0; hd < 8; ++hd) {
          const float p = (hd < G) ? fast_exp2(sv[hd] - ref[hd]) : 0.f;
          const bool bigger = sv[hd] > smax[hd];
          lrest[hd] += bigger ? pmax[hd] : p;
          pmax[hd] = bigger ? p : pmax[hd];
          smax[hd] = fmaxf(smax[hd], sv[hd]);
          pv[hd] = p;
        }
        if (use_base) {
          wait_bounded(&vfull[vs], vpar, &ctl[0], status, wait_cycles, false);
          const float bval = valid ? baseV[vs * kT + tok] : 0.f;
          const bool bigger = bval > bmax;
          brest += bigger ? bmax : bval;
          bmax = bigger ? bval : bmax;
          pv[7] = bval;  // row 7 of P^T carries the base score (G <= 7 here)
        }
        // the P^T buffer is read by the previous product until odone says otherwise
        if (ti >= 1) wait_bounded(odone, (ti - 1) & 1, &ctl[0], status, wait_cycles, false);
#pragma unroll
        for (int hd = 0; hd < 8; hd += 2) {  // rows hd (hi part) and 8 + hd (lo part), column = token
          if (hd < G || (use_base && hd == 6)) {
            const uint32_t hi2 = pack_bf16x2(pv[hd], pv[hd + 1]);
            const uint32_t lo2 = pack_bf16x2(pv[hd] - __uint_as_float(hi2 << 16), pv[hd + 1] - __uint_as_float(hi2 & 0xffff0000u));
            char* at0 = pb_tok + hd * 128 + ((pchunk ^ hd) << 4);
            char* at1 = pb_tok + (hd + 1) * 128 + ((pchunk ^ (hd + 1)) << 4);
            *reinterpret_cast<unsigned short*>(at0) = (unsigned short)(hi2 & 0xffffu);
            *reinterpret_cast<unsigned short*>(at1) = (unsigned short)(hi2 >> 16);
            *reinterpret_cast<unsigned short*>(at0 + 1024) = (unsigned short)(lo2 & 0xffffu);
            *reinterpret_cast<unsigned short*>(at1 + 1024) = (unsigned short)(lo2 >> 16);
          }
        }
        if (n_valid < kT) {
          // rows behind the unit's length hold whatever the cache has there: clear them in the V tile so
          // that a zero weight times a stray NaN cannot reach the accumulators
          wait_bounded(&vfull[vs], vpar, &ctl[0], status, wait_cycles, false);
          if (!valid) {
            char* vt = tilesV + vs * kTileBytes;
#pragma unroll
            for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4*>(vt + tile_off(tok, c)) = make_uint4(0u, 0u, 0u, 0u);
          }
        }
        fence_async_smem();
        prefill::tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(pfull);
      }

      // ===================== close: this CTA's record =====================
      float osum[8];
#pragma unroll
      for (int hd = 0; hd < 8; ++hd) osum[hd] = 0.f;
      if (w.T > 0) {
        wait_bounded(odone, (ti - 1) & 1, &ctl[0], status, wait_cycles, false);
        prefill::tc_fence_after();
        float ov[16];
        tmem_ld16(tO + lane_base, ov);  // lane = channel
        prefill::tc_fence_before();
#pragma unroll
        for (int hd = 0; hd < 8; ++hd) osum[hd] = ov[hd] + ov[8 + hd];
      }
      // (sum of the others, largest, its logit) per head over the warp: three halving steps that also deal
      // the heads out (lanes 16.. keep heads 4..7, and so on), then two plain steps; lane 4 * i ends up
      // with head (i & 1) * 4 + ((i >> 1) & 1) * 2 + (i >> 2)
      {
        const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0, up4 = (lane & 4) != 0;
        float l4[4], p4[4], s4[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float sl = up16 ? lrest[i] : lrest[4 + i], sp = up16 ? pmax[i] : pmax[4 + i], ss = up16 ? smax[i] : smax[4 + i];
          l4[i] = up16 ? lrest[4 + i] : lrest[i]; p4[i] = up16 ? pmax[4 + i] : pmax[i]; s4[i] = up16 ? smax[4 + i] : smax[i];
          top_merge(l4[i], p4[i], s4[i], __shfl_xor_sync(0xffffffffu, sl, 16), __shfl_xor_sync(0xffffffffu, sp, 16),
                    __shfl_xor_sync(0xffffffffu, ss, 16));
        }
        float l2[2], p2[2], s2[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float sl = up8 ? l4[i] : l4[2 + i], sp = up8 ? p4[i] : p4[2 + i], ss = up8 ? s4[i] : s4[2 + i];
          l2[i] = up8 ? l4[2 + i] : l4[i]; p2[i] = up8 ? p4[2 + i] : p4[i]; s2[i] = up8 ? s4[2 + i] : s4[i];
          top_merge(l2[i], p2[i], s2[i], __shfl_xor_sync(0xffffffffu, sl, 8), __shfl_xor_sync(0xffffffffu, sp, 8),
                    __shfl_xor_sync(0xffffffffu, ss, 8));
        }
        float l1, p1, s1;
        {
          const float sl = up4 ? l2[0] : l2[1], sp = up4 ? p2[0] : p2[1], ss = up4 ? s2[0] : s2[1];
          l1 = up4 ? l2[1] : l2[0]; p1 = up4 ? p2[1] : p2[0]; s1 = up4 ? s2[1] : s2[0];
          top_merge(l1, p1, s1, __shfl_xor_sync(0xffffffffu, sl, 4), __shfl_xor_sync(0xffffffffu, sp, 4),
                    __shfl_xor_sync(0xffffffffu, ss, 4));
        }
#pragma unroll
        for (int off = 2; off > 0; off >>= 1)
          top_merge(l1, p1, s1, __shfl_xor_sync(0xffffffffu, l1, off), __shfl_xor_sync(0xffffffffu, p1, off),
                    __shfl_xor_sync(0xffffffffu, s1, off));
        if ((lane & 3) == 0) {
          const int hd = ((lane >> 4) & 1) * 4 + ((lane >> 3) & 1) * 2 + ((lane >> 2) & 1);
          gred[gw * 28 + hd * 3] = l1;
          gred[gw * 28 + hd * 3 + 1] = p1;
          gred[gw * 28 + hd * 3 + 2] = s1;
        }
      }
      // the carried base scores the same way, keyed by their own size
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float ol = __shfl_xor_sync(0xffffffffu, brest, off), op = __shfl_xor_sync(0xffffffffu, bmax, off);
        const bool mine = bmax >= op;
        brest = brest + ol + (mine ? op : bmax);
        bmax = mine ? bmax : op;
      }
      if (lane == 0) {
        gred[gw * 28 + 24] = brest;
        gred[gw * 28 + 25] = bmax;
      }
      group_sync(0);
      // across the four warps (threads 0..8): this CTA's record
      if (tok < 9) {
        float a_l, a_p, a_s = 0.f;
        if (tok < 8) {
          a_l = gred[tok * 3]; a_p = gred[tok * 3 + 1]; a_s = gred[tok * 3 + 2];
#pragma unroll
          for (int ww = 1; ww < 4; ++ww) top_merge(a_l, a_p, a_s, gred[ww * 28 + tok * 3], gred[ww * 28 + tok * 3 + 1], gred[ww * 28 + tok * 3 + 2]);
          float myref = -INFINITY;
#pragma unroll
          for (int hd = 0; hd < 8; ++hd)
            if (tok == hd) myref = ref[hd];
          mystat[tok] = myref;
          mystat[8 + tok] = a_l;
          mystat[16 + tok] = a_p;
          mystat[24 + tok] = a_s;
        } else {
          a_l = gred[24]; a_p = gred[25];
#pragma unroll
          for (int ww = 1; ww < 4; ++ww) {
            const float ol = gred[ww * 28 + 24], op = gred[ww * 28 + 25];
            const bool mine = a_p >= op;
            a_l = a_l + ol + (mine ? op : a_p);
            a_p = mine ? a_p : op;
          }
          mystat[32] = a_l;
          mystat[33] = a_p;
          mystat[34] = 0.f;
          mystat[35] = 0.f;
        }
      }
      // the peers' copies of the previous unit's records must have been read before they are overwritten
      if (mu >= 1) wait_bounded(r2, (mu - 1) & 1, &ctl[0], status, wait_cycles, false);
      group_sync(0);
      if (!ctl[0]) {  // (a CTA that has given up pushes nothing more: its peers may be on their way out)
        // statistics to every peer (one 16-byte piece per thread and peer)
        const uint32_t st_local = smem_u32(xstats + rank * kStatFloats), bar_local = smem_u32(r1);
        for (int p = tok; p < 9 * C; p += kGroup) {
          const int peer = p / 9, piece = p - peer * 9;
          const float4 v = *reinterpret_cast<const float4*>(mystat + piece * 4);
          push_f32x4(map_to_rank(st_local, peer) + piece * 16, v.x, v.y, v.z, v.w, map_to_rank(bar_local, peer));
        }
        // partial outputs (thread = channel) to the owner of the channel: xo[record][channel in slice][head]
        const int owner = tok / slice, cl = tok - owner * slice;
        const int own_nch = min(slice, kD - owner * slice);
        const uint32_t ra = map_to_rank(smem_u32(xo), owner) + (uint32_t)(((rank * own_nch + cl) * 8) * 4);
        const uint32_t rb = map_to_rank(bar_local, owner);
        push_f32x4(ra, osum[0], osum[1], osum[2], osum[3], rb);
        push_f32x4(ra + 16, osum[4], osum[5], osum[6], osum[7], rb);
      }
      ++mu;
    }
  } else {
    // ================================ keeper groups (thread = token of the tile) ================================
    // Group bg takes the CTA's tiles j with j % kNB == bg: it keeps their logits and value rows during the
    // attention pass and scores them after the merge. Both groups finish the softmax statistics for
    // themselves (no hand-over between them); the owner's channels are dealt to them in turn.
    const int bg = (warp >> 2) - 1, gw = warp & 3;
    const int tok = tid & (kGroup - 1);
    const uint32_t lane_base = (uint32_t)(32 * gw) << 16;
    Fin* fin = fins + bg;
    float* fac = facs + bg * kMaxC * 8;
    float keep[kMaxKeep][8];  // this thread's logits (log2 domain) of the unit's tiles it keeps
    float keepb[kMaxKeep];    // and their carried base scores
    int ti = 0;               // tiles this CTA has been through before the current unit
    int mu = 0;               // units merged so far (phases of r1 / r2)

    for (int k = 0; k < nk; ++k) {
      const Work w = sch.at(k);
      if (!w.ok) continue;
      const int b = w.unit / dm.Hkv, h = w.unit % dm.Hkv;

      // ===================== attention pass: keep logits and value rows =====================
#pragma unroll 1
      for (int jj = 0; kNB * jj + bg < w.T; ++jj) {
        const int j = kNB * jj + bg, tj = ti + j;
        const int t = w.t0 + j;
        const int n_valid = min(kT, w.n - t * kT);
        const int vs = tj % kVS, sb = tj % kSB;
        wait_bounded(&sfull[sb], (tj / kSB) & 1, &ctl[0], status, wait_cycles, false);
        prefill::tc_fence_after();
        float sv[8];
        tmem_ld8(tS + lane_base + sb * 16, sv);
        prefill::tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sfree[sb]);
        const bool valid = tok < n_valid;
#pragma unroll
        for (int hd = 0; hd < 8; ++hd) sv[hd] = (valid && hd < G) ? sv[hd] * scale2 : -INFINITY;
        wait_bounded(&vfull[vs], (tj / kVS) & 1, &ctl[0], status, wait_cycles, false);
        const float bval = (use_base && valid) ? baseV[vs * kT + tok] : 0.f;
#pragma unroll
        for (int q = 0; q < kMaxKeep; ++q)  // (static indices keep the arrays in registers)
          if (q == jj) {
#pragma unroll
            for (int hd = 0; hd < 8; ++hd) keep[q][hd] = sv[hd];
            keepb[q] = bval;
          }
        if (j < kStash) {
          const char* vt = tilesV + vs * kTileBytes;
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            uint32_t rw[32];
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const uint4 raw = *reinterpret_cast<const uint4*>(vt + tile_off(tok, half * 8 + c));
              rw[4 * c] = raw.x; rw[4 * c + 1] = raw.y; rw[4 * c + 2] = raw.z; rw[4 * c + 3] = raw.w;
            }
            prefill::tmem_st32u(tStash + lane_base + j * 64 + half * 32, rw);
          }
          prefill::tmem_st_wait();
          __syncwarp();
          if (lane == 0) mbar_arrive(&vempty[vs]);
        }
      }

      // ===================== merge =====================
      wait_bounded(r1, mu & 1, &ctl[0], status, wait_cycles, false);
      {
        // warp gw finishes heads 2 gw and 2 gw + 1: the lower 16 lanes one, the upper 16 the other; lane = record
        const int hd = 2 * gw + (lane >> 4), rl = lane & 15;
        const bool have = rl < C;
        const float* st = xstats + rl * kStatFloats;
        // with carried base scores the eighth half-warp has no head (G <= 7): it merges the base scores instead,
        // (sum of the others, largest) with the score itself as the key, through the same steps
        const bool is_base = use_base && hd == 7;
        const float rc = have ? (is_base ? 0.f : st[hd]) : -INFINITY;
        float m_fin = rc;
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) m_fin = fmaxf(m_fin, __shfl_xor_sync(0xffffffffu, m_fin, off));
        const float f = (rc == -INFINITY) ? 0.f : fast_exp2(rc - m_fin);
        const float lr = have ? (is_base ? st[32] : st[8 + hd] * f) : 0.f, pm = have ? (is_base ? st[33] : st[16 + hd] * f) : 0.f;
        const float sx = have ? (is_base ? st[33] : st[24 + hd]) : -INFINITY;
        float smx = sx;
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) smx = fmaxf(smx, __shfl_xor_sync(0xffffffffu, smx, off));
        const uint32_t bal = (__ballot_sync(0xffffffffu, have && sx == smx) >> (lane & 16)) & 0xffffu;
        const int cstar = __ffs(bal) - 1;
        float lsum = lr + ((rl != cstar) ? pm : 0.f);
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, off);
        const float pmf = __shfl_sync(0xffffffffu, pm, (lane & 16) + max(cstar, 0));
        const float l = lsum + pmf;
        const float inv_l = (hd < G && l > 0.f) ? __fdividef(1.f, l) : 0.f;
        if (rl == 0) {
          fin->m[hd] = (hd < G) ? m_fin + __log2f(l) : 0.f;
          fin->inv_l[hd] = inv_l;
          fin->smax[hd] = smx;
          fin->crest[hd] = lsum * inv_l;
          if (is_base) {
            fin->hbsum = l;
            fin->bmax = smx;
            fin->brest = lsum;
            fin->Htot = (counted ? (float)G : 0.f) + l;
          } else if (!use_base && hd == 0) {
            fin->hbsum = 0.f;
            fin->bmax = 0.f;
            fin->brest = 0.f;
            fin->Htot = (float)G;
          }
        }
        if (have) fac[rl * 8 + hd] = is_base ? 1.f : f * inv_l;
      }
      group_sync(1 + bg);
      {
        // owners: o and -X of this CTA's channels of this group's parity; 8 lanes per channel, lane = head
        const float inv_H = (fin->Htot > 0.f) ? 1.f / fin->Htot : 0.f;
        float* xdst = xnX + (mu & 1) * kD;
        const int r = tok & 7;
        const int nq = (my_nch - bg + kNB - 1) / kNB;  // channels dealt to this group
        for (int q0 = 0; q0 < nq; q0 += kGroup / 8) {
          const int cl = kNB * (q0 + (tok >> 3)) + bg;
          const bool act = cl < my_nch;
          float v0 = 0.f, v1 = 0.f;
          if (act) {
            int c = 0;
            for (; c + 1 < C; c += 2) {
              v0 = fmaf(fac[c * 8 + r], xo[(c * my_nch + cl) * 8 + r], v0);
              v1 = fmaf(fac[c * 8 + 8 + r], xo[((c + 1) * my_nch + cl) * 8 + r], v1);
            }
            if (c < C) v0 = fmaf(fac[c * 8 + r], xo[(c * my_nch + cl) * 8 + r], v0);
          }
          const float val = v0 + v1;
          const bool is_head = act && r < G;
          if (is_head) o[((size_t)b * dm.Hq + h * G + r) * kD + my_ch0 + cl] = val;
          float xs = (is_head && counted) ? val : ((act && use_base && r == 7) ? val : 0.f);
#pragma unroll
          for (int off = 4; off > 0; off >>= 1) xs += __shfl_xor_sync(0xffffffffu, xs, off);
          // FastCAOTE (Sec. 3.3): the distances are taken to the mean of the unit's value rows instead of X
          const float nxv = vsum ? -(act ? __ldg(vsum + (size_t)w.unit * kD + my_ch0 + cl) / (float)w.n : 0.f) : -(xs * inv_H);
          if (act && !ctl[0]) {
            for (int peer = r; peer < C; peer += 8)
              push_f32(map_to_rank(smem_u32(xdst + my_ch0 + cl), peer), nxv, map_to_rank(smem_u32(r2), peer));
          }
        }
      }
      group_sync(1 + bg);  // every thread of this group is done with the records: tell the peers
      if (tok < C && !ctl[0]) push_f32(map_to_rank(smem_u32(xword + kNB * rank + bg), tok), 0.f, map_to_rank(smem_u32(r2), tok));
      wait_bounded(r2, mu & 1, &ctl[0], status, wait_cycles, false);
      if (bg == 0 && tok == 0 && !ctl[0]) {
        // the next unit's merge: what the peers will push into this CTA. (Not after a wait of this CTA has run
        // out: the phase may then still be open, and a second arrival on an open phase whose arrival count is
        // already used up is not defined.)
        mbar_expect_tx(r1, r1_bytes);
        mbar_expect_tx(r2, r2_bytes);
      }

      // ===================== score pass (a held tile first: its V slot is wanted back) =====================
      {
        const float Htot = fin->Htot, hbsum = fin->hbsum, fbmax = fin->bmax, fbrest = fin->brest;
        const float* nX = xnX + (mu & 1) * kD;
        const int mine = (w.T + kNB - 1 - bg) / kNB;                     // tiles this group kept
        const int first_held = (kStash + kNB - 1 - bg) / kNB;            // smallest jj with kNB jj + bg >= kStash
        const int nheld = max(mine - first_held, 0);
#pragma unroll 1
        for (int jx = 0; jx < mine; ++jx) {
          const int jj = (jx < nheld) ? first_held + jx : jx - nheld;
          const int j = kNB * jj + bg;
          const int t = w.t0 + j;
          const int n_valid = min(kT, w.n - t * kT);
          const bool valid = tok < n_valid;
          float sl[8], bold = 0.f;
#pragma unroll
          for (int q = 0; q < kMaxKeep; ++q)
            if (q == jj) {
#pragma unroll
              for (int hd = 0; hd < 8; ++hd) sl[hd] = keep[q][hd];
              bold = keepb[q];
            }
          float asum = 0.f, comp = 0.f;
          if (counted) {
#pragma unroll
            for (int hd = 0; hd < 8; ++hd) {
              if (hd < G) {
                const float a = fast_exp2(sl[hd] - fin->m[hd]);
                asum += a;
                comp += (sl[hd] == fin->smax[hd]) ? fin->crest[hd] : 1.f - a;
              }
            }
          }
          float hj = asum, rest = comp;
          if (use_base) {
            const float bcomp = (bold == fbmax) ? fbrest : hbsum - bold;
            if (mode == CAOTE_BASE_ACCUM) { hj = bold + asum; rest = comp + bcomp; }
            else { hj = bold; rest = bcomp; }
          }
          float2 acc[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) acc[i] = make_float2(0.f, 0.f);
          const int vs = (ti + j) % kVS;
          if (j < kStash) {
            // the row comes back from TMEM in four pieces of 32 channels; the next piece is in flight while
            // this one is used
            uint32_t ra[16], rb[16];
            tmem_ld16u(tStash + lane_base + j * 64, ra);
#pragma unroll
            for (int piece = 0; piece < 4; ++piece) {
              tmem_ld_wait();
              if (piece < 3) {
                if (piece & 1) tmem_ld16u(tStash + lane_base + j * 64 + (piece + 1) * 16, ra);
                else tmem_ld16u(tStash + lane_base + j * 64 + (piece + 1) * 16, rb);
              }
              const uint32_t* rw = (piece & 1) ? rb : ra;
#pragma unroll
              for (int c = 0; c < 16; c += 2) {
                const float4 x = *reinterpret_cast<const float4*>(nX + piece * 32 + 2 * c);
                const float2 d0 = __fadd2_rn(make_float2(__uint_as_float(rw[c] << 16), __uint_as_float(rw[c] & 0xffff0000u)), make_float2(x.x, x.y));
                const float2 d1 = __fadd2_rn(make_float2(__uint_as_float(rw[c + 1] << 16), __uint_as_float(rw[c + 1] & 0xffff0000u)), make_float2(x.z, x.w));
                acc[c & 2] = __ffma2_rn(d0, d0, acc[c & 2]);
                acc[(c & 2) + 1] = __ffma2_rn(d1, d1, acc[(c & 2) + 1]);
              }
            }
          } else {
            const char* vt = tilesV + vs * kTileBytes;
#pragma unroll
            for (int c = 0; c < 16; ++c) {
              const uint4 raw = *reinterpret_cast<const uint4*>(vt + tile_off(tok, c));
              const float4 x0 = *reinterpret_cast<const float4*>(nX + 8 * c);
              const float4 x1 = *reinterpret_cast<const float4*>(nX + 8 * c + 4);
              const float2 d0 = __fadd2_rn(make_float2(__uint_as_float(raw.x << 16), __uint_as_float(raw.x & 0xffff0000u)), make_float2(x0.x, x0.y));
              const float2 d1 = __fadd2_rn(make_float2(__uint_as_float(raw.y << 16), __uint_as_float(raw.y & 0xffff0000u)), make_float2(x0.z, x0.w));
              const float2 d2 = __fadd2_rn(make_float2(__uint_as_float(raw.z << 16), __uint_as_float(raw.z & 0xffff0000u)), make_float2(x1.x, x1.y));
              const float2 d3 = __fadd2_rn(make_float2(__uint_as_float(raw.w << 16), __uint_as_float(raw.w & 0xffff0000u)), make_float2(x1.z, x1.w));
              acc[0] = __ffma2_rn(d0, d0, acc[0]);
              acc[1] = __ffma2_rn(d1, d1, acc[1]);
              acc[2] = __ffma2_rn(d2, d2, acc[2]);
              acc[3] = __ffma2_rn(d3, d3, acc[3]);
            }
          }
          const float n2 = ((acc[0].x + acc[0].y) + (acc[1].x + acc[1].y)) + ((acc[2].x + acc[2].y) + (acc[3].x + acc[3].y));
          if (valid) {
            const size_t slot = (size_t)w.unit * dm.cap + (size_t)t * kT + tok;
            if (mode == CAOTE_BASE_ACCUM) base[slot] = hj;
            float sc = 0.f;
            if (Htot > 0.f && hj > 0.f) sc = (rest > 0.f) ? __fdividef(hj, rest) * fast_sqrt(n2) : INFINITY;
            scores[slot] = sc;
          }
          if (j >= kStash) {
            __syncwarp();
            if (lane == 0) mbar_arrive(&vempty[vs]);
          }
        }
      }
      // the heads' log-sum-exp, left for the post-eviction output (alpha_j = 2^(s_j - m)); off the merge's path
      if (bg == 0 && rank == 0 && tok < G) {
        float* hs = reinterpret_cast<float*>(reinterpret_cast<char*>(status) + kHeaderBytes) + (size_t)w.unit * kHeadStatFloats;
        hs[tok] = fin->m[tok];
        hs[8 + tok] = fin->smax[tok];
        hs[16 + tok] = fin->crest[tok];
      }
      ti += w.T;
      ++mu;
    }
  }

  // Leave only after every copy this CTA issued has landed and every peer is done with this CTA's shared
  // memory, whatever the reason for leaving.
  prefill::tc_fence_before();
  __syncthreads();
  prefill::tc_fence_after();
  if (ctl[0]) {
    if (tid == 0)
      for (int s = 0; s < kKS; ++s) {
        // the newest copy into each slot: issue number i with i % kKS == s
        const int issued = ctl[1];
        const int i = issued - 1 - ((issued - 1 - s) % kKS + kKS) % kKS;
        if (issued > 0 && i >= 0 && !mbar_try_wait(&kfull[s], (i / kKS) & 1)) drain_wait(&kfull[s], (i / kKS) & 1, status);
      }
    if (tid == 32)
      for (int s = 0; s < kVS; ++s) {
        const int issued = ctl[2];
        const int i = issued - 1 - ((issued - 1 - s) % kVS + kVS) % kVS;
        if (issued > 0 && i >= 0 && !mbar_try_wait(&vfull[s], (i / kVS) & 1)) drain_wait(&vfull[s], (i / kVS) & 1, status);
      }
    __syncthreads();
  }
  if (warp == kWarpQK) prefill::tmem_dealloc(tmem, kTmemCols);
  cluster_sync_all();
}

}  // namespace dcl
}  // namespace caote
