// Greedy multi-token eviction (Appendix B of the paper, the two-token derivation chained) with a unit's value rows
// resident on chip: a thread-block cluster per (sequence, KV head) unit, every CTA holding a contiguous share of the
// unit's value rows in its shared memory (bf16, head_dim 128). Each pick sweeps those rows from shared memory instead
// of from L2 (the one-CTA kernel in greedy.cuh re-reads all of them from L2 for every pick):
//   every CTA: distances of its rows to the current output X = Y / H, its best (score bits, position) candidate;
//   every CTA stores its candidate and the candidate's value row into every CTA's shared memory (distributed shared
//   memory stores: nobody waits for them); one cluster barrier; every CTA takes the same minimum of the candidates it
//   now holds and updates its own copy of Y and H with the winner's row (the same arithmetic everywhere, so the
//   copies never differ). Reading the candidates and then the row from their owners after the barrier cost two more
//   round trips through distributed shared memory per pick.
// The candidates are double-buffered by the parity of the pick, which is what makes one barrier per pick enough.
// A CTA holds up to kMaxRows rows in shared memory; a unit too long for 16 CTAs' worth leaves the rest of every CTA's
// share in global memory, and the CTA sweeps that part from L2 (several rows in flight per warp): still 16 SMs
// pulling on a sixteenth each instead of one SM on all of it.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace caote {
namespace greedy_cl {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr int kD = 128;
constexpr int kMaxRows = 768;   // value rows per CTA in shared memory (192 KB)
constexpr int kMaxShare = 2048; // rows per CTA in all (the weights and distances of all of them are in shared memory)
constexpr int kMaxC = 16;

struct Cand {  // a CTA's best candidate of a pick
  unsigned long long key;  // (score bits << 32) | position
  int slot;                // slot in the unit, -1: none
  float h;                 // its weight
};

inline size_t smem_bytes(int rows_smem, int rows) {
  return (size_t)rows_smem * kD * 2 + sizeof(float) * (2 * (size_t)rows + kD + (kD + 4) + 2 * kWarps) +
         sizeof(unsigned long long) * kWarps + sizeof(int) * (2 * kWarps + 8) + 64;
}

__device__ __forceinline__ uint32_t gc_rank() { return ptx::cluster_ctarank(); }
__device__ __forceinline__ uint32_t gc_size() { return ptx::cluster_nctarank(); }
__device__ __forceinline__ uint32_t gc_cluster_id() { return ptx::cluster_id_x(); }
__device__ __forceinline__ void gc_sync() { ptx::cluster_sync_all(); }
// The same shared-memory location in the CTA of rank `rank`.
__device__ __forceinline__ uint32_t gc_map(const void* p, uint32_t rank) { return ptx::map_to_rank(ptx::smem_u32(p), rank); }
__device__ __forceinline__ float gc_ld_f32(uint32_t a) { return ptx::ld_dsmem_f32(a); }
__device__ __forceinline__ int gc_ld_s32(uint32_t a) { return ptx::ld_dsmem_s32(a); }

// grid = units x C CTAs in clusters of C; rows_per = rows of the unit per CTA (the same for every CTA of the grid),
// the first rows_smem of them in shared memory.
__global__ void __launch_bounds__(kThreads, 1)
greedy_cluster_kernel(int Hkv, int cap, int rows_per, int rows_smem, const __nv_bfloat16* __restrict__ V, const float* __restrict__ h_in,
                      const int* __restrict__ len, const int* __restrict__ budget, const int* __restrict__ pos,
                      int* __restrict__ evict_idx, int* __restrict__ order_out, int max_evict, int* __restrict__ n_evict,
                      int* status) {
  extern __shared__ __align__(16) unsigned char gsm[];
  __nv_bfloat16* Vs = reinterpret_cast<__nv_bfloat16*>(gsm);            // [rows_smem][kD]
  float* hs = reinterpret_cast<float*>(Vs + (size_t)rows_smem * kD);    // [rows_per] weight, < 0 once evicted
  float* ds = hs + rows_per;                                            // [rows_per] || X - v_j || of the current state
  float* Ys = ds + rows_per;                                            // [kD] sum of h_j v_j over the tokens present
  float* part = Ys + kD;                                                // [kD + 4] this CTA's share of Y and (at kD) of H
  float* wsum = part + kD + 4;                                          // [2 * kWarps]
  unsigned long long* wkey = reinterpret_cast<unsigned long long*>(wsum + 2 * kWarps);  // [kWarps]
  int* wslot = reinterpret_cast<int*>(wkey + kWarps);                   // [2 * kWarps]
  int* misc = wslot + 2 * kWarps;                                       // [8]: 0 count of evicted rows here, 1 running count
  __shared__ float s_H, s_he;
  __shared__ int s_e;
  __shared__ __align__(16) Cand pcand[2][kMaxC];                 // [parity of the pick][rank]: every CTA's candidate
  __shared__ __align__(16) __nv_bfloat16 prow[2][kMaxC][kD];     // ... and its value row

  const int C = (int)gc_size(), rank = (int)gc_rank();
  const int unit = (int)gc_cluster_id(), b = unit / Hkv, hd = unit % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = len[b];
  int bud = budget[b];
  if (bud < 1) bud = 1;
  int k = n - bud;
  if (k < 0 || n > cap) k = 0;
  if (k > max_evict) {
    if (tid == 0 && rank == 0) set_status(status, CAOTE_ERR_OVERFLOW);
    k = 0;
  }
  if (hd == 0 && rank == 0 && tid == 0) n_evict[b] = k;
  if (k == 0) return;  // (the whole cluster leaves: no barrier is outstanding)
  const int r0 = rank * rows_per;
  const int nr = max(0, min(rows_per, n - r0));  // rows of the unit this CTA holds
  const __nv_bfloat16* Vu = V + ((size_t)unit * cap + r0) * kD;
  const float* hu = h_in + (size_t)unit * cap + r0;
  const int* pu = pos ? pos + (size_t)unit * cap + r0 : nullptr;
  int* out = evict_idx + (size_t)unit * max_evict;
  int* ord = order_out ? order_out + (size_t)unit * max_evict : nullptr;

  // ---- the rows into shared memory; H and Y of this CTA's rows (fixed order of the partial sums) ----
  const int ns = min(nr, rows_smem);  // rows held in shared memory; rows [ns, nr) stay in global memory
  for (int i = tid; i < ns * (kD / 8); i += kThreads)
    reinterpret_cast<uint4*>(Vs)[i] = reinterpret_cast<const uint4*>(Vu)[i];
  float hsum = 0.f;
  for (int j = tid; j < nr; j += kThreads) {
    const float hj = fmaxf(hu[j], 0.f);
    hs[j] = hj;
    hsum += hj;
  }
  hsum = warp_sum(hsum);
  if (lane == 0) wsum[warp] = hsum;
  __syncthreads();
  float yacc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int j = warp; j < nr; j += kWarps) {
    const float hj = hs[j];
    const uint2 raw = *reinterpret_cast<const uint2*>((j < ns ? Vs : Vu) + (size_t)j * kD + 4 * lane);
    yacc[0] = fmaf(hj, __uint_as_float(raw.x << 16), yacc[0]);
    yacc[1] = fmaf(hj, __uint_as_float(raw.x & 0xffff0000u), yacc[1]);
    yacc[2] = fmaf(hj, __uint_as_float(raw.y << 16), yacc[2]);
    yacc[3] = fmaf(hj, __uint_as_float(raw.y & 0xffff0000u), yacc[3]);
  }
  if (tid < kD + 4) part[tid] = 0.f;
  __syncthreads();
  for (int w = 0; w < kWarps; ++w) {  // warps add their parts one after the other: reproducible
    if (warp == w) {
#pragma unroll
      for (int c = 0; c < 4; ++c) part[4 * lane + c] += yacc[c];
    }
    __syncthreads();
  }
  if (tid == 0) {
    float H = 0.f;
    for (int w = 0; w < kWarps; ++w) H += wsum[w];
    part[kD] = H;
    misc[0] = 0;
  }
  gc_sync();  // every CTA's share is written
  if (tid <= kD) {  // the unit's Y and H: the shares in rank order, the same sum in every CTA
    float tot = 0.f;
    for (int i = 0; i < C; ++i) tot += gc_ld_f32(gc_map(part + tid, (uint32_t)i));
    if (tid < kD) Ys[tid] = tot; else s_H = tot;
  }
  __syncthreads();

  for (int t = 0; t < k; ++t) {
    const float H = s_H;
    const float inv_H = (H > 0.f) ? 1.f / H : 0.f;
    // ---- distances of this CTA's tokens still present to the current output: four tokens per warp at a time, eight
    //      lanes per token (channels [8 l, 8 l + 8) and [64 + 8 l, 64 + 8 l + 8): both 16-byte loads of a token are
    //      contiguous over its lanes), three shuffle steps per sum; a warp per token with five steps spent most of the
    //      sweep waiting for its own shuffles ----
    {
      const int sub = lane >> 3, l8 = lane & 7;
      float xa[8], xb[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        xa[c] = Ys[8 * l8 + c] * inv_H;
        xb[c] = Ys[64 + 8 * l8 + c] * inv_H;
      }
      for (int j0 = 4 * warp; j0 < ns; j0 += 4 * kWarps) {
        const int j = j0 + sub;
        const bool live = j < ns && hs[j] >= 0.f;
        float acc = 0.f;
        if (live) {
          const uint4 ra = *reinterpret_cast<const uint4*>(Vs + (size_t)j * kD + 8 * l8);
          const uint4 rb = *reinterpret_cast<const uint4*>(Vs + (size_t)j * kD + 64 + 8 * l8);
          const uint32_t wa[4] = {ra.x, ra.y, ra.z, ra.w}, wb[4] = {rb.x, rb.y, rb.z, rb.w};
          float acc2 = 0.f;
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float a0 = xa[2 * c] - __uint_as_float(wa[c] << 16), a1 = xa[2 * c + 1] - __uint_as_float(wa[c] & 0xffff0000u);
            const float b0 = xb[2 * c] - __uint_as_float(wb[c] << 16), b1 = xb[2 * c + 1] - __uint_as_float(wb[c] & 0xffff0000u);
            acc = fmaf(a0, a0, fmaf(a1, a1, acc));
            acc2 = fmaf(b0, b0, fmaf(b1, b1, acc2));
          }
          acc += acc2;
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 4);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        if (live && l8 == 0) ds[j] = sqrtf(acc);
      }
    }
    // ... and of the rows it left in global memory, the same way with four passes' loads in flight per warp
    {
      constexpr int kPasses = 4;
      const int sub = lane >> 3, l8 = lane & 7;
      float xa[8], xb[8];
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        xa[c] = Ys[8 * l8 + c] * inv_H;
        xb[c] = Ys[64 + 8 * l8 + c] * inv_H;
      }
      for (int j0 = ns + 4 * warp; j0 < nr; j0 += 4 * kWarps * kPasses) {
        uint4 ra[kPasses], rb[kPasses];
        bool live[kPasses];
#pragma unroll
        for (int u = 0; u < kPasses; ++u) {
          const int j = j0 + u * 4 * kWarps + sub;
          live[u] = j < nr && hs[j] >= 0.f;
          if (live[u]) {
            ra[u] = *reinterpret_cast<const uint4*>(Vu + (size_t)j * kD + 8 * l8);
            rb[u] = *reinterpret_cast<const uint4*>(Vu + (size_t)j * kD + 64 + 8 * l8);
          }
        }
#pragma unroll
        for (int u = 0; u < kPasses; ++u) {
          float acc = 0.f;
          if (live[u]) {
            const uint32_t wa[4] = {ra[u].x, ra[u].y, ra[u].z, ra[u].w}, wb[4] = {rb[u].x, rb[u].y, rb[u].z, rb[u].w};
            float acc2 = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float a0 = xa[2 * c] - __uint_as_float(wa[c] << 16), a1 = xa[2 * c + 1] - __uint_as_float(wa[c] & 0xffff0000u);
              const float b0 = xb[2 * c] - __uint_as_float(wb[c] << 16), b1 = xb[2 * c + 1] - __uint_as_float(wb[c] & 0xffff0000u);
              acc = fmaf(a0, a0, fmaf(a1, a1, acc));
              acc2 = fmaf(b0, b0, fmaf(b1, b1, acc2));
            }
            acc += acc2;
          }
          acc += __shfl_xor_sync(0xffffffffu, acc, 4);
          acc += __shfl_xor_sync(0xffffffffu, acc, 2);
          acc += __shfl_xor_sync(0xffffffffu, acc, 1);
          if (live[u] && l8 == 0) ds[j0 + u * 4 * kWarps + sub] = sqrtf(acc);
        }
      }
    }
    __syncthreads();
    // ---- this CTA's arg-min of w_j / (1 - w_j) * dist_j over (score bits, position) (a thread per token; doing
    //      this inside the sweep, with the division and the position load on every warp's path, was slower) ----
    unsigned long long best = ~0ull;
    int best_slot = -1;
    for (int j = tid; j < nr; j += kThreads) {
      const float hj = hs[j];
      if (hj < 0.f) continue;
      float sc = 0.f;
      if (H > 0.f && hj > 0.f) {
        const float rest = H - hj;  // the others' weight (times H)
        sc = (rest > 0.f) ? hj / rest * ds[j] : INFINITY;
      }
      const unsigned long long key = ((unsigned long long)__float_as_uint(sc) << 32) | (unsigned int)(pu ? pu[j] : r0 + j);
      if (key < best) { best = key; best_slot = j; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
      const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
      if (ok < best || (ok == best && os >= 0 && (best_slot < 0 || os < best_slot))) { best = ok; best_slot = os; }
    }
    if (lane == 0) { wkey[warp] = best; wslot[warp] = best_slot; }
    __syncthreads();
    // every warp reduces the warps' results for itself: this CTA's candidate (local slot bs, -1: none)
    unsigned long long bk = lane < kWarps ? wkey[lane] : ~0ull;
    int bs = lane < kWarps ? wslot[lane] : -1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok = __shfl_xor_sync(0xffffffffu, bk, o);
      const int os = __shfl_xor_sync(0xffffffffu, bs, o);
      if (os >= 0 && (bs < 0 || ok < bk || (ok == bk && os < bs))) { bk = ok; bs = os; }
    }
    // ---- the candidate and its value row go to every CTA of the cluster (this one included) ----
    const int par = t & 1;
    if (tid < 16 * C) {  // 16 bytes of the row per thread, 16 threads per peer
      const int peer = tid >> 4, chunk = tid & 15;
      if (bs >= 0) {
        const uint4 v = *reinterpret_cast<const uint4*>((bs < ns ? Vs : Vu) + (size_t)bs * kD + 8 * chunk);
        ptx::st_dsmem_v4(gc_map(&prow[par][rank][8 * chunk], (uint32_t)peer), v);
      }
    } else if (tid >= 256 && tid < 256 + C) {
      uint4 cd;
      cd.x = (uint32_t)bk;
      cd.y = (uint32_t)(bk >> 32);
      cd.z = (uint32_t)(bs >= 0 ? r0 + bs : -1);
      cd.w = __float_as_uint(bs >= 0 ? hs[bs] : 0.f);
      ptx::st_dsmem_v4(gc_map(&pcand[par][rank], (uint32_t)(tid - 256)), cd);
    }
    gc_sync();  // every CTA's candidate of this pick has arrived (and everybody is done with the pick before)
    // ---- the unit's pick: the smallest candidate, lower slot on equal keys; the same in every CTA ----
    if (warp == 0) {
      unsigned long long ck = ~0ull;
      int cs = -1;
      float ch = 0.f;
      if (lane < C) {
        const Cand rc = pcand[par][lane];
        cs = rc.slot;
        ck = rc.key;
        ch = rc.h;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xffffffffu, ck, o);
        const int os = __shfl_xor_sync(0xffffffffu, cs, o);
        const float oh = __shfl_xor_sync(0xffffffffu, ch, o);
        if (os >= 0 && (cs < 0 || ok < ck || (ok == ck && os < cs))) { ck = ok; cs = os; ch = oh; }
      }
      if (lane == 0) { s_e = cs; s_he = ch; }
    }
    __syncthreads();
    const int e = s_e;
    if (e < 0) break;  // (cannot happen with k < n; the same in every CTA, so no barrier is left unmatched)
    // ---- evict e: Y -= h_e v_e, H -= h_e (the row came with its owner's candidate) ----
    const float he = s_he;
    const int owner = e / rows_per, el = e - owner * rows_per;
    if (tid < kD) Ys[tid] -= he * __bfloat162float(prow[par][owner][tid]);
    if (tid == 0) {
      s_H = H - he;
      if (ord && rank == 0) ord[t] = e;
      if (owner == rank) {
        hs[el] = -1.f;
        misc[0] += 1;
      }
    }
    __syncthreads();
  }
  // ---- the evicted slots in ascending order (the layout caote_compact expects): CTAs in rank order ----
  gc_sync();  // every CTA's count of evicted rows is final
  if (tid == 0) {
    int before = 0;
    for (int i = 0; i < rank; ++i) before += gc_ld_s32(gc_map(misc, (uint32_t)i));
    misc[1] = before;
  }
  __syncthreads();
  for (int j0 = 0; j0 < nr; j0 += kThreads) {
    const int j = j0 + tid;
    const bool gone = j < nr && hs[j] < 0.f;
    const unsigned m = __ballot_sync(0xffffffffu, gone);
    if (lane == 0) wslot[kWarps + warp] = __popc(m);
    __syncthreads();
    int at = misc[1];
    for (int w = 0; w < warp; ++w) at += wslot[kWarps + w];
    if (gone) out[at + __popc(m & ((1u << lane) - 1u))] = r0 + j;
    __syncthreads();
    if (tid == 0) {
      int tot = misc[1];
      for (int w = 0; w < kWarps; ++w) tot += wslot[kWarps + w];
      misc[1] = tot;
    }
    __syncthreads();
  }
  gc_sync();  // no CTA leaves while a peer may still read its shared memory
}

}  // namespace greedy_cl
}  // namespace caote
