// Single-query (decode) scoring path, bf16, head_dim 128, group size <= 8: one thread-block cluster per
// (sequence, KV head) unit, K and V read from HBM exactly once.
//
// Why a cluster. The score c_j = w_j / (1 - w_j) * ||X - v_j|| needs every value row twice: once for
// the attention output (which gives X) and once more, after X is known, for the distance. A unit's
// cluster keeps the value rows on chip between the two uses, so the second use costs no HBM traffic:
//   * the unit's 128-token tiles are dealt to the C CTAs of the cluster (at most kMaxT each);
//   * attention pass: K and V tiles stream through two TMA rings; S^T = K_tile Q^T and
//     O^T += V_tile^T P^T run on tcgen05 with the tile's tokens on the M side (a token owns one TMEM
//     lane and one thread); right after its V tile has landed the token's thread copies its own value
//     row (256 bytes) into a TMEM stash slot (64 columns per tile, 7 slots beside the accumulators); a
//     CTA's tiles beyond the 7th stay in their V ring slot instead; the token's logits stay in registers;
//   * merge: every CTA pushes its (reference, sums, partial output) record to its peers through
//     distributed shared memory (st.async, completion counted by an mbarrier of the receiver): the
//     softmax statistics go to everyone, the partial outputs to the CTA that owns the channel slice;
//     the owners finish o and X for their channels and push X to everyone (two rounds in all);
//   * score pass: every thread takes its tokens' rows back from the stash, forms ||X - v_j||^2 by
//     plain subtraction and writes c_j.
// Nothing but q, K, V, base are read from global memory and nothing but o, scores, base is written.
//
// 1 - w_j without cancellation (Sec. 3.2 normalisation; a token that holds almost all the weight): per
// head the largest numerator is kept apart from the sum of the others, through the thread, the group,
// the CTA and the cluster, so that the complement of the head's top token is l_rest / l (a sum of the
// other tokens' numerators) and every other token's complement is 1 - alpha with alpha <= 1/2; the
// carried base scores are treated the same way. The heads' complements, all non-negative, are added.
//
// Warp roles (384 threads): warps 0..3 and 4..7 are two token groups that take the CTA's tiles in turn
// (each with its own S^T and O^T accumulators and P^T buffer); one lane each of warps 8..11 issues the
// K copies, the V copies, the S^T products and the O^T products.
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
constexpr int kStash = 7;                 // value tiles a CTA keeps in TMEM
constexpr int kMaxT = 9;                  // tiles of one unit per CTA: the stash + 2 held in the V ring
constexpr int kMaxKeep = (kMaxT + 1) / 2; // tiles of one unit per token group
constexpr int kMaxC = 16;                 // largest cluster
constexpr int kGroup = 128;               // threads of a token group
constexpr int kThreads = 2 * kGroup + 128;
constexpr int kWarpK = 8, kWarpV = 9, kWarpQK = 10, kWarpPV = 11;
constexpr int kQBufBytes = 2048;          // 8 query rows x 128 channels as two 64-channel boxes
constexpr int kPBytes = 4096;             // 16 rows x 128 tokens as two 64-token boxes
constexpr int kStatFloats = 36;           // per (CTA, group): ref[8] lrest[8] pmax[8] smax[8] brest bmax pad pad
constexpr int kXoBytes = 9216;            // partial outputs received: [2C][8][slice] floats, slice = ceil(128 / C)
constexpr int kLenTab = 512;              // unit lengths of this cluster kept in shared memory
constexpr uint32_t kTmemCols = 512;       // S^T x 2, O^T x 2 (16 columns each), 7 stash slots of 64 columns
constexpr long long kDrainCycles = 4000000000LL;  // waits for hardware to finish what was already issued

struct Fin {        // per unit, every CTA computes its own copy
  float m[8];       // final softmax reference per head (log2 domain)
  float inv_l[8];   // 1 / sum_j 2^(s_j - m)
  float smax[8];    // largest logit of the head
  float crest[8];   // (sum of the numerators of all tokens but the head's top one) / l
  float Htot;       // normaliser of the base score
  float hbsum;      // sum of the carried base scores
  float bmax;       // largest carried base score
  float brest;      // sum of the other carried base scores
};

inline size_t smem_bytes() {
  return 1024 + (size_t)(kKS + kVS) * kTileBytes + 2 * kQBufBytes + 2 * kPBytes + kVS * (kT * 4) +
         2 * kMaxC * kStatFloats * 4 + kXoBytes + kD * 4 + sizeof(Fin) + 2 * kMaxC * 8 * 4 /* fac */ +
         2 * 64 * 4 /* red */ + 2 * 4 * 28 * 4 /* gred */ + kLenTab * 4 + 40 * 8 /* barriers */ + 64;
}

// ---- cluster PTX ------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_id_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_count_x() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
  return r;
}
// Address of the same shared-memory location in the CTA of rank `rank` of this cluster.
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
// One float into a peer's shared memory; the peer's mbarrier counts the 4 bytes when they have landed.
__device__ __forceinline__ void push_f32(uint32_t remote_addr, float v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(remote_addr), "r"(__float_as_uint(v)), "r"(remote_bar) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Wait for hardware to finish what has already been issued (copies in flight, queued products).
__device__ __forceinline__ void drain_wait(uint64_t* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    __nanosleep(50);
    if (clock64() - t0 > kDrainCycles) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      return;
    }
  }
}
// Bounded wait; a wait that runs out records the timeout and raises the stop flag. Never blocks once the
// flag is up.
__device__ __forceinline__ void wait_bounded(uint64_t* bar, uint32_t parity, volatile int* stop, int* status,
                                             long long limit, bool idle) {
  if (*stop || mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (idle) __nanosleep(20);
    if (*stop) return;
    if (clock64() - t0 > limit) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      *stop = 1;
      return;
    }
  }
}
// Barrier of one token group (ids 1 and 2), with and without an OR-reduction.
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
__device__ __forceinline__ void groups_sync() { asm volatile("bar.sync 3, %0;" ::"n"(2 * kGroup) : "memory"); }

__device__ __forceinline__ void tmem_ld32u(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 16; A K-major or MN-major, B K-major.
using decode::idesc_n16;
// k-step ks of the query operand: two boxes of 8 rows x 128 bytes, 1024 bytes apart. The product reads 16
// rows (N = 16); rows 8..15 fall on whatever follows in shared memory and only feed unused columns.
__device__ __forceinline__ uint64_t desc_q(uint32_t addr, int ks) {
  return prefill::smem_desc(addr + (ks >> 2) * 1024 + (ks & 3) * 32, 16, 1024);
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

__global__ void __launch_bounds__(kThreads, 1)
decode_cluster_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                      const __grid_constant__ CUtensorMap tmQ, Dims dm, const int* __restrict__ len,
                      float* __restrict__ base, float* __restrict__ o, float* __restrict__ scores, int* status,
                      long long wait_cycles) {
  extern __shared__ char smem_raw[];
  char* sm = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  char* tilesK = sm;                                                   // [kKS][kTileBytes]
  char* tilesV = tilesK + kKS * kTileBytes;                            // [kVS][kTileBytes]
  char* qbuf = tilesV + kVS * kTileBytes;                              // [2][kQBufBytes]
  char* pbuf = qbuf + 2 * kQBufBytes;                                  // [2 groups][kPBytes]
  float* baseV = reinterpret_cast<float*>(pbuf + 2 * kPBytes);         // [kVS][kT] carried base scores of a V slot's tile
  float* xstats = baseV + kVS * kT;                                    // [2C][kStatFloats]   written by the peers
  float* xo = xstats + 2 * kMaxC * kStatFloats;                        // [2C][8][slice]      written by the peers
  float* xX = xo + kXoBytes / 4;                                       // [kD]                written by the owners
  Fin* fin = reinterpret_cast<Fin*>(xX + kD);
  float* fac = reinterpret_cast<float*>(fin + 1);                      // [2C][8] 2^(ref_c - m) / l per record and head
  float* red = fac + 2 * kMaxC * 8;                                    // [2 groups][2][4][8] warp maxima
  float* gred = red + 2 * 64;                                          // [2 groups][4 warps][28] closing sums
  int* slen = reinterpret_cast<int*>(gred + 2 * 4 * 28);               // [kLenTab]
  uint64_t* bars = reinterpret_cast<uint64_t*>(slen + kLenTab);
  uint64_t* kfull = bars;                 // [kKS]
  uint64_t* kempty = kfull + kKS;         // [kKS]   the S^T product has read the slot
  uint64_t* vfull = kempty + kKS;         // [kVS]
  uint64_t* vempty = vfull + kVS;         // [kVS]   4 warps of the tile's group + the O^T product
  uint64_t* sfull = vempty + kVS;         // [2]     S^T of the group's tile is formed
  uint64_t* sfree = sfull + 2;            // [2]     the group has read it (4 warps)
  uint64_t* pfull = sfree + 2;            // [2]     P^T of the group's tile is written (4 warps)
  uint64_t* odone = pfull + 2;            // [2]     O^T += of the group's tile is done
  uint64_t* qfree = odone + 2;            // [2]     the last S^T product of the unit that used the buffer is done
  uint64_t* r1 = qfree + 2;               // records of all (CTA, group) pairs have landed
  uint64_t* r2 = r1 + 1;                  // X has landed
  uint64_t* done_bar = r2 + 1;            // [2]     every product of an issuer has finished
  volatile int* ctl = reinterpret_cast<volatile int*>(done_bar + 2);   // [0] stop, [1] K copies issued, [2] V copies issued
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(const_cast<int*>(ctl) + 4);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = dm.G, mode = dm.base_mode;
  const bool use_base = (mode == CAOTE_BASE_ACCUM || mode == CAOTE_BASE_EXTERNAL);
  const bool counted = (mode != CAOTE_BASE_EXTERNAL);
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

  if (tid == 0) {
    for (int i = 0; i < kKS; ++i) { mbar_init(&kfull[i], 1); mbar_init(&kempty[i], 1); }
    for (int i = 0; i < kVS; ++i) { mbar_init(&vfull[i], 1); mbar_init(&vempty[i], 5); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sfull[i], 1);
      mbar_init(&sfree[i], 4);
      mbar_init(&pfull[i], 4);
      mbar_init(&odone[i], 1);
      mbar_init(&qfree[i], 1);
      mbar_init(&done_bar[i], 1);
    }
    mbar_init(r1, 1);
    mbar_init(r2, 1);
    ctl[0] = 0;
    ctl[1] = 0;
    ctl[2] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int k = tid; k < min(nk, kLenTab); k += kThreads) slen[k] = __ldg(len + (sch.cid + k * sch.ncl) / dm.Hkv);
  // rows of P^T that no head writes stay zero for the whole kernel
  for (int i = tid; i < 2 * kPBytes / 16; i += kThreads) reinterpret_cast<uint4*>(pbuf)[i] = make_uint4(0u, 0u, 0u, 0u);
  fence_async_smem();
  if (warp == kWarpQK) prefill::tmem_alloc(tmem_slot, kTmemCols);
  prefill::tc_fence_before();
  __syncthreads();
  prefill::tc_fence_after();
  cluster_sync_all();  // every peer's barriers exist before anyone pushes to them
  const uint32_t tmem = *tmem_slot;
  const uint32_t tS = tmem, tO = tmem + 32, tStash = tmem + 64;

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
      int ki = 0, us = 0, cs[2] = {0, 0};
      for (int k = 0; k < nk && !ctl[0]; ++k) {
        const Work w = sch.at(k);
        if (!w.ok || w.T == 0) continue;
        const uint32_t qa = smem_u32(qbuf + (us & 1) * kQBufBytes);
        for (int j = 0; j < w.T; ++j) {
          const int g = j & 1, s = ki % kKS;
          wait_bounded(&kfull[s], (ki / kKS) & 1, &ctl[0], status, wait_cycles, true);
          if (cs[g] >= 1) wait_bounded(&sfree[g], (cs[g] - 1) & 1, &ctl[0], status, wait_cycles, true);
          if (ctl[0]) break;
          prefill::tc_fence_after();
          const uint32_t ka = smem_u32(tilesK + s * kTileBytes);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            prefill::umma(tS + g * 16, prefill::desc_k_major(ka, ks), desc_q(qa, ks), kIdQK, ks > 0);
          prefill::umma_commit(&sfull[g]);
          prefill::umma_commit(&kempty[s]);
          if (j == w.T - 1) prefill::umma_commit(&qfree[us & 1]);
          ++ki;
          ++cs[g];
        }
        ++us;
      }
      // nothing of this CTA's may still be running in the tensor pipe when TMEM is given back
      prefill::umma_commit(&done_bar[0]);
      drain_wait(&done_bar[0], 0, status);
    }
  } else if (warp == kWarpPV) {
    // ================================ O^T products (one lane) ================================
    if (lane == 0) {
      constexpr uint32_t kIdPV = idesc_n16(true);
      int vi = 0, cp[2] = {0, 0};
      for (int k = 0; k < nk && !ctl[0]; ++k) {
        const Work w = sch.at(k);
        if (!w.ok) continue;
        for (int j = 0; j < w.T; ++j) {
          const int g = j & 1, s = vi % kVS;
          wait_bounded(&vfull[s], (vi / kVS) & 1, &ctl[0], status, wait_cycles, true);
          wait_bounded(&pfull[g], cp[g] & 1, &ctl[0], status, wait_cycles, false);
          if (ctl[0]) break;
          prefill::tc_fence_after();
          const uint32_t va = smem_u32(tilesV + s * kTileBytes);
          const uint32_t pa = smem_u32(pbuf + g * kPBytes);
          const bool first = j < 2;  // the group's first tile of this unit starts a new sum
#pragma unroll
          for (int kk = 0; kk < 8; ++kk)
            prefill::umma(tO + g * 16, prefill::desc_mn_major(va, kk), decode::desc_rows16(pa, kk), kIdPV, !(first && kk == 0));
          prefill::umma_commit(&odone[g]);
          prefill::umma_commit(&vempty[s]);
          ++vi;
          ++cp[g];
        }
      }
      prefill::umma_commit(&done_bar[1]);
      drain_wait(&done_bar[1], 0, status);
    }
  } else {
    // ================================ token groups (thread = token of the group's tile) ================================
    const int g = warp >> 2, gw = warp & 3;
    const int tok = tid & (kGroup - 1);
    const uint32_t lane_base = (uint32_t)(32 * gw) << 16;
    float* redg = red + g * 64;
    float* gredg = gred + g * 4 * 28;
    char* pb_tok = pbuf + g * kPBytes + (tok >> 6) * 2048 + (tok & 7) * 2;
    const int pchunk = (tok & 63) >> 3;

    float keep[kMaxKeep][8];  // this thread's logits (log2 domain) of the unit's tiles it owns
    float keepb[kMaxKeep];    // and their carried base scores
    int cs = 0;               // tiles this group has been through (phases of sfull / pfull / odone)
    int mu = 0;               // units merged so far (phases of r1 / r2)
    int vi_base = 0;          // V tiles of this CTA before the current unit
    int red_par = 0;

    for (int k = 0; k < nk; ++k) {
      const Work w = sch.at(k);
      if (!w.ok) {
        if (w.n != 0 && tid == 0 && rank == 0) set_status(status, CAOTE_ERR_BAD_LENGTH);
        continue;
      }
      const int b = w.unit / dm.Hkv, h = w.unit % dm.Hkv;
      float ref[8], lrest[8], pmax[8], smax[8];
      float brest = 0.f, bmax = 0.f;
#pragma unroll
      for (int hd = 0; hd < 8; ++hd) { ref[hd] = -INFINITY; lrest[hd] = 0.f; pmax[hd] = 0.f; smax[hd] = -INFINITY; }
      if (tid == 0) {
        // this unit's merge: what the peers will push into this CTA
        mbar_expect_tx(r1, (uint32_t)(2 * C * (kStatFloats * 4 + 8 * my_nch * 4)));
        mbar_expect_tx(r2, (uint32_t)(kD * 4));
      }

      // ===================== attention pass over this group's tiles =====================
#pragma unroll 1
      for (int jj = 0; jj < kMaxKeep; ++jj) {
        const int j = 2 * jj + g;
        if (j < w.T) {
          const int t = w.t0 + j;
          const int n_valid = min(kT, w.n - t * kT);
          const int vi = vi_base + j, vs = vi % kVS;
          const uint32_t vpar = (vi / kVS) & 1;
          const bool first = (jj == 0);
          wait_bounded(&sfull[g], cs & 1, &ctl[0], status, wait_cycles, false);
          prefill::tc_fence_after();
          float sv[8];
          tmem_ld8(tS + lane_base + g * 16, sv);
          prefill::tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sfree[g]);
          const bool valid = tok < n_valid;
          bool over = false;
#pragma unroll
          for (int hd = 0; hd < 8; ++hd) {
            sv[hd] = (valid && hd < G) ? sv[hd] * scale2 : -INFINITY;
            over |= sv[hd] > ref[hd] + 8.f;
          }
#pragma unroll
          for (int q = 0; q < kMaxKeep; ++q)  // (static indices keep the array in registers)
            if (q == jj) {
#pragma unroll
              for (int hd = 0; hd < 8; ++hd) keep[q][hd] = sv[hd];
            }
          float bval = 0.f;
          if (use_base) {
            wait_bounded(&vfull[vs], vpar, &ctl[0], status, wait_cycles, false);
            bval = valid ? baseV[vs * kT + tok] : 0.f;
          }
#pragma unroll
          for (int q = 0; q < kMaxKeep; ++q)
            if (q == jj) keepb[q] = bval;
          if (group_any(g, over)) {
            // a logit tops its head's reference by more than 2^8 (always on the group's first tile): move
            // the references to the maxima seen so far and rescale what has been accumulated
            float* rd = redg + red_par * 32;
            red_par ^= 1;
#pragma unroll
            for (int hd = 0; hd < 8; ++hd) {
              if (hd < G) {
                const float mx = warp_max(sv[hd]);
                if (lane == 0) rd[gw * 8 + hd] = mx;
              }
            }
            group_sync(g);
            float corr[8];
            bool changed = false;
#pragma unroll
            for (int hd = 0; hd < 8; ++hd) {
              corr[hd] = 1.f;
              if (hd < G) {
                const float nr = fmaxf(fmaxf(ref[hd], fmaxf(rd[hd], rd[8 + hd])), fmaxf(rd[16 + hd], rd[24 + hd]));
                corr[hd] = fast_exp2(ref[hd] - nr);  // 2^-inf = 0 on the group's first tile
                changed |= nr != ref[hd];
                lrest[hd] *= corr[hd];
                pmax[hd] *= corr[hd];
                ref[hd] = nr;
              }
            }
            if (!first && changed) {
              // O^T of the tiles so far (lane = channel); the group's previous product must have finished
              wait_bounded(&odone[g], (cs - 1) & 1, &ctl[0], status, wait_cycles, false);
              prefill::tc_fence_after();
              float ov[16];
              tmem_ld16(tO + lane_base + g * 16, ov);
#pragma unroll
              for (int hd = 0; hd < 8; ++hd) { ov[hd] *= corr[hd]; ov[8 + hd] *= corr[hd]; }
              tmem_st16(tO + lane_base + g * 16, ov);
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
            pv[hd] = (use_base && hd == 7) ? bval : p;
          }
          {
            const bool bigger = bval > bmax;
            brest += bigger ? bmax : bval;
            bmax = bigger ? bval : bmax;
          }
          // the group's P^T buffer is read by its previous product until odone says otherwise
          if (cs >= 1) wait_bounded(&odone[g], (cs - 1) & 1, &ctl[0], status, wait_cycles, false);
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
          char* vt = tilesV + vs * kTileBytes;
          if (n_valid < kT) {
            // rows behind the unit's length hold whatever the cache has there: clear them in the V tile so
            // that a zero weight times a stray NaN cannot reach the accumulators
            wait_bounded(&vfull[vs], vpar, &ctl[0], status, wait_cycles, false);
            if (!valid) {
#pragma unroll
              for (int c = 0; c < 16; ++c) *reinterpret_cast<uint4*>(vt + tile_off(tok, c)) = make_uint4(0u, 0u, 0u, 0u);
            }
          }
          fence_async_smem();
          prefill::tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(&pfull[g]);
          // keep the token's value row: into the TMEM stash, or (tiles beyond the stash) where it is
          wait_bounded(&vfull[vs], vpar, &ctl[0], status, wait_cycles, false);
          if (j < kStash) {
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
          ++cs;
        }
      }

      // ===================== close: this group's record =====================
      const int my_tiles = (w.T + 1 - g) / 2;
      float osum[8];
#pragma unroll
      for (int hd = 0; hd < 8; ++hd) osum[hd] = 0.f;
      if (my_tiles > 0) {
        wait_bounded(&odone[g], (cs - 1) & 1, &ctl[0], status, wait_cycles, false);
        prefill::tc_fence_after();
        float ov[16];
        tmem_ld16(tO + lane_base + g * 16, ov);  // lane = channel
        prefill::tc_fence_before();
#pragma unroll
        for (int hd = 0; hd < 8; ++hd) osum[hd] = ov[hd] + ov[8 + hd];
      }
      // (sum of the others, largest, its logit) per head over the group's threads: first inside a warp
#pragma unroll
      for (int hd = 0; hd < 8; ++hd) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          const float ol = __shfl_xor_sync(0xffffffffu, lrest[hd], off);
          const float op = __shfl_xor_sync(0xffffffffu, pmax[hd], off);
          const float os = __shfl_xor_sync(0xffffffffu, smax[hd], off);
          const bool mine = smax[hd] >= os;
          lrest[hd] = lrest[hd] + ol + (mine ? op : pmax[hd]);
          pmax[hd] = mine ? pmax[hd] : op;
          smax[hd] = fmaxf(smax[hd], os);
        }
        if (lane == 0) {
          gredg[gw * 28 + hd * 3] = lrest[hd];
          gredg[gw * 28 + hd * 3 + 1] = pmax[hd];
          gredg[gw * 28 + hd * 3 + 2] = smax[hd];
        }
      }
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        const float ol = __shfl_xor_sync(0xffffffffu, brest, off);
        const float op = __shfl_xor_sync(0xffffffffu, bmax, off);
        const bool mine = bmax >= op;
        brest = brest + ol + (mine ? op : bmax);
        bmax = mine ? bmax : op;
      }
      if (lane == 0) {
        gredg[gw * 28 + 24] = brest;
        gredg[gw * 28 + 25] = bmax;
      }
      group_sync(g);
      const uint32_t rec = (uint32_t)(2 * rank + g);
      // then across the group's four warps (threads 0..8), pushed to every peer
      if (tok < 9) {
        float a_l, a_p, a_s = 0.f;
        if (tok < 8) {
          a_l = gredg[tok * 3]; a_p = gredg[tok * 3 + 1]; a_s = gredg[tok * 3 + 2];
#pragma unroll
          for (int ww = 1; ww < 4; ++ww) {
            const float ol = gredg[ww * 28 + tok * 3], op = gredg[ww * 28 + tok * 3 + 1], os = gredg[ww * 28 + tok * 3 + 2];
            const bool mine = a_s >= os;
            a_l = a_l + ol + (mine ? op : a_p);
            a_p = mine ? a_p : op;
            a_s = fmaxf(a_s, os);
          }
        } else {
          a_l = gredg[24]; a_p = gredg[25];
#pragma unroll
          for (int ww = 1; ww < 4; ++ww) {
            const float ol = gredg[ww * 28 + 24], op = gredg[ww * 28 + 25];
            const bool mine = a_p >= op;
            a_l = a_l + ol + (mine ? op : a_p);
            a_p = mine ? a_p : op;
          }
        }
        float myref = -INFINITY;
#pragma unroll
        for (int hd = 0; hd < 8; ++hd)
          if (tok == hd) myref = ref[hd];
        const uint32_t st_local = smem_u32(xstats + rec * kStatFloats);
        const uint32_t bar_local = smem_u32(r1);
        for (int peer = 0; peer < C; ++peer) {
          const uint32_t ra = map_to_rank(st_local, peer), rb = map_to_rank(bar_local, peer);
          if (tok < 8) {
            push_f32(ra + (tok) * 4, myref, rb);
            push_f32(ra + (8 + tok) * 4, a_l, rb);
            push_f32(ra + (16 + tok) * 4, a_p, rb);
            push_f32(ra + (24 + tok) * 4, a_s, rb);
          } else {
            push_f32(ra + 32 * 4, a_l, rb);
            push_f32(ra + 33 * 4, a_p, rb);
            push_f32(ra + 34 * 4, 0.f, rb);
            push_f32(ra + 35 * 4, 0.f, rb);
          }
        }
      }
      {
        // partial outputs (thread = channel) to the owner of the channel: xo[rec][head][channel in slice]
        const int owner = tok / slice, cl = tok - owner * slice;
        const int own_nch = min(slice, kD - owner * slice);
        const uint32_t ra = map_to_rank(smem_u32(xo), owner) + (uint32_t)((rec * 8 * own_nch + cl) * 4);
        const uint32_t rb = map_to_rank(smem_u32(r1), owner);
#pragma unroll
        for (int hd = 0; hd < 8; ++hd) push_f32(ra + (uint32_t)(hd * own_nch * 4), osum[hd], rb);
      }

      // ===================== merge =====================
      wait_bounded(r1, mu & 1, &ctl[0], status, wait_cycles, false);
      {
        // warp `warp` (0..7) finishes head `warp`; lane = record
        const int hd = warp;
        const bool have = lane < 2 * C;
        const float* st = xstats + lane * kStatFloats;
        const float rc = have ? st[hd] : -INFINITY;
        const float m_fin = warp_max(rc);
        const float f = (rc == -INFINITY) ? 0.f : exp2f(rc - m_fin);
        const float lr = have ? st[8 + hd] * f : 0.f, pm = have ? st[16 + hd] * f : 0.f;
        const float sx = have ? st[24 + hd] : -INFINITY;
        const float smx = warp_max(sx);
        const int cstar = __ffs(__ballot_sync(0xffffffffu, have && sx == smx)) - 1;
        const float lsum = warp_sum(lr + ((lane != cstar) ? pm : 0.f));
        const float pmf = __shfl_sync(0xffffffffu, pm, max(cstar, 0));
        const float l = lsum + pmf;
        const float inv_l = (hd < G && l > 0.f) ? 1.f / l : 0.f;
        if (lane == 0) {
          fin->m[hd] = (hd < G) ? m_fin : 0.f;
          fin->inv_l[hd] = inv_l;
          fin->smax[hd] = smx;
          fin->crest[hd] = lsum * inv_l;
        }
        if (have) fac[lane * 8 + hd] = (use_base && hd == 7) ? 1.f : f * inv_l;
        if (hd == 7) {
          // carried base scores: largest one apart from the sum of the others
          const float bm = have ? st[33] : 0.f, br = have ? st[32] : 0.f;
          const float bmx = warp_max(bm);
          const int bstar = __ffs(__ballot_sync(0xffffffffu, have && bm == bmx)) - 1;
          const float brs = warp_sum(br + ((lane != bstar) ? bm : 0.f));
          if (lane == 0) {
            const float hbsum = use_base ? brs + bmx : 0.f;
            fin->hbsum = hbsum;
            fin->bmax = bmx;
            fin->brest = brs;
            fin->Htot = (counted ? (float)G : 0.f) + hbsum;
          }
        }
      }
      groups_sync();
      {
        // owners: o and X of this CTA's channels; 16 lanes per channel, lane = head (8..15 idle)
        const float Htot = fin->Htot;
        const int lim = (16 * my_nch + 31) & ~31;
        for (int p = tid; p < lim; p += 2 * kGroup) {
          const int cl = p >> 4, r = p & 15;
          const bool act = cl < my_nch && r < 8;
          float val = 0.f;
          if (act) {
            for (int c = 0; c < 2 * C; ++c) val = fmaf(fac[c * 8 + r], xo[(c * 8 + r) * my_nch + cl], val);
          }
          const bool is_head = act && r < G;
          if (is_head) o[((size_t)b * dm.Hq + h * G + r) * kD + my_ch0 + cl] = val;
          float xs = (is_head && counted) ? val : ((act && use_base && r == 7) ? val : 0.f);
#pragma unroll
          for (int off = 8; off > 0; off >>= 1) xs += __shfl_xor_sync(0xffffffffu, xs, off);
          const float xv = (Htot > 0.f) ? xs / Htot : 0.f;
          if (cl < my_nch && r < C)
            push_f32(map_to_rank(smem_u32(xX + my_ch0 + cl), r), xv, map_to_rank(smem_u32(r2), r));
        }
      }
      wait_bounded(r2, mu & 1, &ctl[0], status, wait_cycles, false);

      // ===================== score pass over this group's tiles =====================
      {
        const float Htot = fin->Htot, hbsum = fin->hbsum, fbmax = fin->bmax, fbrest = fin->brest;
#pragma unroll 1
        for (int jj = 0; jj < kMaxKeep; ++jj) {
          const int j = 2 * jj + g;
          if (j < w.T) {
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
                  const float s = sl[hd];
                  const float a = fast_exp2(s - fin->m[hd]) * fin->inv_l[hd];
                  asum += a;
                  comp += (s == fin->smax[hd]) ? fin->crest[hd] : 1.f - a;
                }
              }
            }
            float hj = asum, rest = comp;
            if (use_base) {
              const float bcomp = (bold == fbmax) ? fbrest : hbsum - bold;
              if (mode == CAOTE_BASE_ACCUM) { hj = bold + asum; rest = comp + bcomp; }
              else { hj = bold; rest = bcomp; }
            }
            float n2a = 0.f, n2b = 0.f;
            const int vs = (vi_base + j) % kVS;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              uint32_t rw[32];
              if (j < kStash) {
                tmem_ld32u(tStash + lane_base + j * 64 + half * 32, rw);
              } else {
                const char* vt = tilesV + vs * kTileBytes;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                  const uint4 raw = *reinterpret_cast<const uint4*>(vt + tile_off(tok, half * 8 + c));
                  rw[4 * c] = raw.x; rw[4 * c + 1] = raw.y; rw[4 * c + 2] = raw.z; rw[4 * c + 3] = raw.w;
                }
              }
#pragma unroll
              for (int c = 0; c < 32; c += 2) {
                const float4 x = *reinterpret_cast<const float4*>(xX + half * 64 + 2 * c);
                const float d0 = x.x - __uint_as_float(rw[c] << 16), d1 = x.y - __uint_as_float(rw[c] & 0xffff0000u);
                const float d2 = x.z - __uint_as_float(rw[c + 1] << 16), d3 = x.w - __uint_as_float(rw[c + 1] & 0xffff0000u);
                n2a = fmaf(d0, d0, n2a); n2b = fmaf(d1, d1, n2b);
                n2a = fmaf(d2, d2, n2a); n2b = fmaf(d3, d3, n2b);
              }
            }
            if (valid) {
              const size_t slot = (size_t)w.unit * dm.cap + (size_t)t * kT + tok;
              if (mode == CAOTE_BASE_ACCUM) base[slot] = hj;
              float sc = 0.f;
              if (Htot > 0.f && hj > 0.f) sc = (rest > 0.f) ? hj / rest * sqrtf(n2a + n2b) : INFINITY;
              scores[slot] = sc;
            }
            if (j >= kStash) {
              __syncwarp();
              if (lane == 0) mbar_arrive(&vempty[vs]);
            }
          }
        }
      }
      vi_base += w.T;
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
        if (issued > 0 && i >= 0) drain_wait(&kfull[s], (i / kKS) & 1, status);
      }
    if (tid == 32)
      for (int s = 0; s < kVS; ++s) {
        const int issued = ctl[2];
        const int i = issued - 1 - ((issued - 1 - s) % kVS + kVS) % kVS;
        if (issued > 0 && i >= 0) drain_wait(&vfull[s], (i / kVS) & 1, status);
      }
    __syncthreads();
  }
  if (warp == kWarpQK) prefill::tmem_dealloc(tmem, kTmemCols);
  cluster_sync_all();
}

}  // namespace dcl
}  // namespace caote
