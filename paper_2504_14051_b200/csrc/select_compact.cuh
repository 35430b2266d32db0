// Selection of the tokens to evict (block radix-select on the bit patterns of the non-negative fp32
// scores, ties broken by original position), in-place compaction of the cache, and the append of new
// tokens. These are bandwidth-trivial next to the scoring pass: n * 4 bytes per unit for selection,
// at most k rows per unit for FILL compaction.
#pragma once

#include "common.cuh"
#include "ptx.cuh"
#include "fast.cuh"

namespace caote {
namespace sel {

constexpr int kSelThreads = 1024;
constexpr int kMaxSharedPicks = 2048;

// 64-bit sort key: score bits in the high word (scores are >= +0, so the unsigned order of the bit
// patterns is the numeric order; +inf sorts last), original position in the low word.
__device__ __forceinline__ unsigned long long make_key(float score, int pos) {
  return ((unsigned long long)__float_as_uint(score) << 32) | (unsigned int)pos;
}

// One CTA per unit. k = max(0, n - budget). Finds the k-th smallest key by 8 passes of an 8-bit
// radix histogram (most significant digit first), then writes the slots whose key is <= that key in
// ascending slot order with a block-wide ordered compaction. (Scores of one unit share their leading bytes, but grouping a
// warp's lanes by digit before the shared-memory atomics, by match_any or by ballots, costs more than the atomics do.)
// Returns k, the number of slots the unit evicts (the same value in every thread of the CTA). With e_smem (room for
// kMaxSharedPicks slots) the chosen slots are also left there when k fits, for a compaction in the same kernel.
__device__ __forceinline__ int select_unit(int unit, int Hkv, int cap, const float* __restrict__ scores,
                                           const int* __restrict__ len, const int* __restrict__ budget,
                                           const int* __restrict__ pos, int* __restrict__ evict_idx, int max_evict,
                                           int* __restrict__ n_evict, int* status, int* e_smem = nullptr) {
  __shared__ unsigned int hist[256];
  __shared__ unsigned long long s_prefix;
  __shared__ int s_remaining;
  __shared__ int s_warp_tot[kSelThreads / 32];
  __shared__ int s_running;
  __shared__ unsigned long long s_min[kSelThreads / 32];

  const int b = unit / Hkv, h = unit % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = len[b];
  int bud = budget[b];
  if (bud < 1) bud = 1;
  int k = n - bud;
  if (k < 0) k = 0;
  if (n > cap) k = 0;
  if (k > max_evict) {
    if (tid == 0) set_status(status, CAOTE_ERR_OVERFLOW);
    k = 0;
  }
  if (h == 0 && tid == 0) n_evict[b] = k;
  if (k == 0) return 0;
  const float* sc = scores + (size_t)unit * cap;
  const int* ps = pos ? pos + (size_t)unit * cap : nullptr;
  int* out = evict_idx + (size_t)unit * max_evict;

  if (k == 1) {  // argmin
    unsigned long long best = ~0ull;
    int best_slot = 0;
    for (int j = tid; j < n; j += kSelThreads) {
      const unsigned long long key = make_key(sc[j], ps ? ps[j] : j);
      if (key < best) { best = key; best_slot = j; }
    }
    // reduce (key, slot): keys are unique when pos is, else the lower slot wins
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
      const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
      if (ok < best || (ok == best && os < best_slot)) { best = ok; best_slot = os; }
    }
    if (lane == 0) { s_min[warp] = best; s_warp_tot[warp] = best_slot; }
    __syncthreads();
    if (warp == 0) {
      best = s_min[lane];
      best_slot = s_warp_tot[lane];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
        const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
        if (ok < best || (ok == best && os < best_slot)) { best = ok; best_slot = os; }
      }
      if (lane == 0) out[0] = best_slot;
    }
    return 1;
  }

  // Radix select on the 64-bit keys, 8 bits per pass, most significant first. Up to kCached keys per
  // thread stay in registers across the passes; a pass ends the search early when the whole bucket it
  // lands in is needed (always the case once the remaining bits only tell equal scores apart and
  // positions are unique).
  constexpr int kCached = 8;
  const bool cached = n <= kSelThreads * kCached;
  unsigned long long kreg[kCached];
#pragma unroll
  for (int i = 0; i < kCached; ++i) {
    const int j = tid + i * kSelThreads;
    kreg[i] = (cached && j < n) ? make_key(sc[j], ps ? ps[j] : j) : ~0ull;
  }
  __shared__ int s_done;
  if (tid == 0) { s_prefix = 0ull; s_remaining = k; s_done = 0; }
  unsigned long long kth = ~0ull;
  for (int pass = 0; pass < 8; ++pass) {
    const int shift = 56 - 8 * pass;
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const unsigned long long prefix = s_prefix;
    const unsigned long long mask = (pass == 0) ? 0ull : (~0ull << (shift + 8));
    if (cached) {
#pragma unroll
      for (int i = 0; i < kCached; ++i) {
        const int j = tid + i * kSelThreads;
        if (j < n && (kreg[i] & mask) == prefix) atomicAdd(&hist[(unsigned int)(kreg[i] >> shift) & 255u], 1u);
      }
    } else {
      for (int j = tid; j < n; j += kSelThreads) {
        const unsigned long long key = make_key(sc[j], ps ? ps[j] : j);
        if ((key & mask) == prefix) atomicAdd(&hist[(unsigned int)(key >> shift) & 255u], 1u);
      }
    }
    __syncthreads();
    if (warp == 0) {
      // the first digit whose cumulative count reaches the number still wanted: 8 bins per lane
      unsigned int c[8], sum = 0u;
#pragma unroll
      for (int q = 0; q < 8; ++q) { c[q] = hist[8 * lane + q]; sum += c[q]; }
      unsigned int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      const unsigned int rem = (unsigned int)s_remaining;
      const unsigned int reach = __ballot_sync(0xffffffffu, rem <= incl);
      const int f = reach ? __ffs((int)reach) - 1 : 31;
      if (lane == f) {
        unsigned int r = rem - (incl - sum);
        int q = 0;
        for (; q < 7; ++q) {
          if (r <= c[q]) break;
          r -= c[q];
        }
        s_remaining = (int)r;
        s_prefix = prefix | ((unsigned long long)(8 * lane + q) << shift);
        s_done = (r == c[q]) ? 1 : 0;
      }
    }
    __syncthreads();
    if (s_done || pass == 7) {
      kth = s_prefix | (shift ? ((1ull << shift) - 1ull) : 0ull);  // the largest key that is taken
      break;
    }
  }
  int* picks = (e_smem && k <= kMaxSharedPicks) ? e_smem : nullptr;
  if (cached) {
    // one scan over the (round, warp) counts, which is the ascending order of the slots tid + round * kSelThreads
    __shared__ int s_cnt[kCached * (kSelThreads / 32)];
    unsigned int ballots[kCached];
#pragma unroll
    for (int i = 0; i < kCached; ++i) {
      const int j = tid + i * kSelThreads;
      ballots[i] = __ballot_sync(0xffffffffu, j < n && kreg[i] <= kth);
      if (lane == 0) s_cnt[i * (kSelThreads / 32) + warp] = __popc(ballots[i]);
    }
    __syncthreads();
    if (warp == 0) {
      constexpr int kPerLane = kCached * (kSelThreads / 32) / 32;
      int c[kPerLane], sum = 0;
#pragma unroll
      for (int q = 0; q < kPerLane; ++q) { c[q] = s_cnt[kPerLane * lane + q]; sum += c[q]; }
      int incl = sum;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
      }
      int run = incl - sum;
#pragma unroll
      for (int q = 0; q < kPerLane; ++q) { s_cnt[kPerLane * lane + q] = run; run += c[q]; }
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < kCached; ++i) {
      if (ballots[i] >> lane & 1u) {
        const int idx = s_cnt[i * (kSelThreads / 32) + warp] + __popc(ballots[i] & ((1u << lane) - 1u));
        if (idx < k) {
          out[idx] = tid + i * kSelThreads;
          if (picks) picks[idx] = tid + i * kSelThreads;
        }
      }
    }
    return k;
  }
  if (tid == 0) s_running = 0;
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += kSelThreads) {
    const int j = j0 + tid;
    const unsigned long long key = (j < n) ? make_key(sc[j], ps ? ps[j] : j) : ~0ull;
    const int flag = (j < n) && (key <= kth);
    const unsigned int ballot = __ballot_sync(0xffffffffu, flag);
    const int in_warp = __popc(ballot & ((1u << lane) - 1u));
    if (lane == 0) s_warp_tot[warp] = __popc(ballot);
    __syncthreads();
    int before = s_running;
    for (int w = 0; w < warp; ++w) before += s_warp_tot[w];
    const int idx = before + in_warp;
    if (flag && idx < k) {
      out[idx] = j;
      if (picks) picks[idx] = j;
    }
    __syncthreads();
    if (tid == 0) {
      int tot = s_running;
      for (int w = 0; w < kSelThreads / 32; ++w) tot += s_warp_tot[w];
      s_running = tot;
    }
    __syncthreads();
  }
  return k;
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(int Hkv, int cap, const float* __restrict__ scores, const int* __restrict__ len,
              const int* __restrict__ budget, const int* __restrict__ pos, int* __restrict__ evict_idx,
              int max_evict, int* __restrict__ n_evict, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  select_unit(blockIdx.x, Hkv, cap, scores, len, budget, pos, evict_idx, max_evict, n_evict, status);
}

// Copy one row of `bytes` bytes (a multiple of 16, 16-byte aligned on both sides) with one warp.
__device__ __forceinline__ void warp_copy_row(char* dst, const char* src, int bytes, int lane) {
  for (int o = lane * 16; o < bytes; o += 32 * 16)
    *reinterpret_cast<uint4*>(dst + o) = *reinterpret_cast<const uint4*>(src + o);
}

// First index in sorted a[0..n) whose value is >= x.
__device__ __forceinline__ int lower_bound(const int* a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a[mid] < x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// FILL compaction, one CTA per unit. With n' = n - k, the evicted slots below n' are holes, and the
// k slots [n', n) hold exactly as many survivors; the i-th surviving tail slot moves into the i-th
// hole. Sources lie in [n', n) and destinations in [0, n'), so no move can clobber another's source.
// E = the unit's k evicted slots in ascending order (global or shared memory). Rows of up to 256 bytes are moved by
// half a warp each, K and V together.
__device__ __forceinline__ void compact_fill_unit(int unit, int k, int Hkv, int cap, int row_bytes, char* __restrict__ K,
                                                  char* __restrict__ V, float* __restrict__ base, int* __restrict__ pos,
                                                  const int* __restrict__ len, const int* E) {
  const int b = unit / Hkv;
  if (k <= 0) return;
  const int n = len[b], n_new = n - k;
  const int nh = lower_bound(E, k, n_new);  // holes = E[0..nh)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int glanes = (row_bytes <= 256) ? 16 : 32;  // lanes that share a row
  const int gl = lane & (glanes - 1);
  const int group = warp * (32 / glanes) + lane / glanes, ngroups = nwarps * (32 / glanes);
  for (int t = group; t < k; t += ngroups) {
    const int s = n_new + t;
    const int lb = nh + lower_bound(E + nh, k - nh, s);
    if (lb < k && E[lb] == s) continue;  // this tail slot is itself evicted
    const int rank = t - (lb - nh);      // its rank among the surviving tail slots
    const int dst = E[rank];
    const size_t so = ((size_t)unit * cap + s), dof = ((size_t)unit * cap + dst);
    if (row_bytes <= 512) {
      if (gl * 16 < row_bytes) {
        const uint4 kr = *reinterpret_cast<const uint4*>(K + so * row_bytes + gl * 16);
        const uint4 vr = *reinterpret_cast<const uint4*>(V + so * row_bytes + gl * 16);
        *reinterpret_cast<uint4*>(K + dof * row_bytes + gl * 16) = kr;
        *reinterpret_cast<uint4*>(V + dof * row_bytes + gl * 16) = vr;
      }
    } else {
      warp_copy_row(K + dof * row_bytes, K + so * row_bytes, row_bytes, lane);
      warp_copy_row(V + dof * row_bytes, V + so * row_bytes, row_bytes, lane);
    }
    if (gl == 0) {
      if (base) base[dof] = base[so];
      if (pos) pos[dof] = pos[so];
    }
  }
}

__global__ void __launch_bounds__(256)
compact_fill_kernel(int Hkv, int cap, int row_bytes, char* __restrict__ K, char* __restrict__ V,
                    float* __restrict__ base, int* __restrict__ pos, const int* __restrict__ len,
                    const int* __restrict__ evict_idx, int max_evict, const int* __restrict__ n_evict) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  compact_fill_unit(blockIdx.x, n_evict[blockIdx.x / Hkv], Hkv, cap, row_bytes, K, V, base, pos, len,
                    evict_idx + (size_t)blockIdx.x * max_evict);
}

// A unit that evicts exactly one token, with FILL compaction: the argmin over (score bits, position) and the move of
// the unit's last row into the hole in one go. The first scores of every thread are fetched before the length is known
// (slots below cap always exist), the last row of K and V is fetched while the scores are searched, and the pick never
// travels through global memory. Same results as select_unit + compact_fill_unit. Returns false, with nothing
// written, unless the unit evicts exactly one token (row_bytes <= 512).
__device__ __forceinline__ bool select_one_fill_unit(int unit, int Hkv, int cap, int row_bytes,
                                                     const float* __restrict__ scores, char* __restrict__ K,
                                                     char* __restrict__ V, float* __restrict__ base,
                                                     int* __restrict__ pos, const int* __restrict__ len,
                                                     const int* __restrict__ budget, int* __restrict__ evict_idx,
                                                     int max_evict, int* __restrict__ n_evict, float* __restrict__ vsum,
                                                     int elt_bytes) {
  __shared__ unsigned long long s_key[kSelThreads / 32];
  __shared__ int s_slot[kSelThreads / 32];
  constexpr int kPer = 8;
  const int b = unit / Hkv, h = unit % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* sc = scores + (size_t)unit * cap;
  const int* ps = pos ? pos + (size_t)unit * cap : nullptr;
  float sv[kPer];
  int pv[kPer];
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int j = tid + i * kSelThreads;
    sv[i] = (j < cap) ? sc[j] : 0.f;
    pv[i] = (ps && j < cap) ? ps[j] : j;
  }
  const int n = len[b];
  int bud = budget[b];
  if (bud < 1) bud = 1;
  if (n > cap || n - bud != 1) return false;
  if (h == 0 && tid == 0) n_evict[b] = 1;
  const int last = n - 1;
  const size_t tail = (size_t)unit * cap + last;
  const bool row_lane = lane * 16 < row_bytes;
  uint4 row = make_uint4(0u, 0u, 0u, 0u);
  float tail_base = 0.f;
  int tail_pos = 0;
  if (warp == 1 && row_lane) row = *reinterpret_cast<const uint4*>(K + tail * row_bytes + lane * 16);
  if (warp == 2 && row_lane) row = *reinterpret_cast<const uint4*>(V + tail * row_bytes + lane * 16);
  if (warp == 3 && lane == 0) {
    if (base) tail_base = base[tail];
    if (pos) tail_pos = pos[tail];
  }
  unsigned long long best = ~0ull;
  int best_slot = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int j = tid + i * kSelThreads;
    const unsigned long long key = make_key(sv[i], pv[i]);
    if (j < n && key < best) { best = key; best_slot = j; }
  }
  for (int j = tid + kPer * kSelThreads; j < n; j += kSelThreads) {
    const unsigned long long key = make_key(sc[j], ps ? ps[j] : j);
    if (key < best) { best = key; best_slot = j; }
  }
  // (key, slot): keys are unique when pos is, else the lower slot wins
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
    const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
    if (ok < best || (ok == best && os < best_slot)) { best = ok; best_slot = os; }
  }
  if (lane == 0) { s_key[warp] = best; s_slot[warp] = best_slot; }
  __syncthreads();
  best = s_key[lane];  // every warp reduces the 32 partial results for itself
  best_slot = s_slot[lane];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
    const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
    if (ok < best || (ok == best && os < best_slot)) { best = ok; best_slot = os; }
  }
  if (tid == 0) evict_idx[(size_t)unit * max_evict] = best_slot;
  if (vsum) {  // FastCAOTE: the evicted row leaves the running sum of values before the last row lands on it
    const int D = row_bytes / elt_bytes, c = tid - 128;
    if (c >= 0 && c < D) {
      const char* vrow = V + ((size_t)unit * cap + best_slot) * row_bytes;
      const float v = (elt_bytes == 2) ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(vrow)[c])
                                       : reinterpret_cast<const float*>(vrow)[c];
      vsum[(size_t)unit * D + c] -= v;
    }
    __syncthreads();
  }
  if (best_slot != last) {  // the last row fills the hole
    const size_t hole = (size_t)unit * cap + best_slot;
    if (warp == 1 && row_lane) *reinterpret_cast<uint4*>(K + hole * row_bytes + lane * 16) = row;
    if (warp == 2 && row_lane) *reinterpret_cast<uint4*>(V + hole * row_bytes + lane * 16) = row;
    if (warp == 3 && lane == 0) {
      if (base) base[hole] = tail_base;
      if (pos) pos[hole] = tail_pos;
    }
  }
  return true;
}

// The CTA that finishes last (a ticket counter, which it also resets) takes the evicted counts off the lengths.
__device__ __forceinline__ void finish_lengths(int B, int* __restrict__ len, const int* __restrict__ n_evict, int* ticket) {
  __shared__ int s_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = (atomicAdd(ticket, 1) == (int)gridDim.x - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int b = threadIdx.x; b < B; b += blockDim.x) len[b] -= __ldcg(&n_evict[b]);
    if (threadIdx.x == 0) *ticket = 0;
  }
}

// Selection and FILL compaction of one unit per CTA in one launch, and the length update by whichever
// CTA finishes last (a ticket counter in the workspace header, which that CTA also resets). Same results
// as select_kernel + compact_fill_kernel + update_len_kernel.
__global__ void __launch_bounds__(kSelThreads)
select_compact_kernel(int B, int Hkv, int cap, int row_bytes, const float* __restrict__ scores, char* __restrict__ K,
                      char* __restrict__ V, float* __restrict__ base, int* __restrict__ pos, int* __restrict__ len,
                      const int* __restrict__ budget, int* __restrict__ evict_idx, int max_evict,
                      int* __restrict__ n_evict, int* status, int* ticket, float* __restrict__ vsum, int elt_bytes) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  const int unit = blockIdx.x;
  if (row_bytes <= 512 &&
      select_one_fill_unit(unit, Hkv, cap, row_bytes, scores, K, V, base, pos, len, budget, evict_idx, max_evict, n_evict,
                           vsum, elt_bytes)) {
    finish_lengths(B, len, n_evict, ticket);
    return;
  }
  __shared__ int s_picks[kMaxSharedPicks];
  const int k = select_unit(unit, Hkv, cap, scores, len, budget, pos, evict_idx, max_evict, n_evict, status, s_picks);
  __syncthreads();  // the unit's picks are written
  // (read back from shared memory where they fit: the searches below are chains of dependent reads)
  const int* E = (k <= kMaxSharedPicks && k > 1) ? s_picks : evict_idx + (size_t)unit * max_evict;
  if (vsum && k > 0) {  // FastCAOTE: the evicted rows leave the running sum of values before they are overwritten
    if (elt_bytes == 2) fast::vsum_sub_unit<__nv_bfloat16>(unit, k, cap, row_bytes / 2, (const __nv_bfloat16*)V, E, vsum);
    else fast::vsum_sub_unit<float>(unit, k, cap, row_bytes / 4, (const float*)V, E, vsum);
    __syncthreads();
  }
  compact_fill_unit(unit, k, Hkv, cap, row_bytes, K, V, base, pos, len, E);
  finish_lengths(B, len, n_evict, ticket);
}

// STABLE compaction: survivors keep their order. grid = (units, 3): y = 0 moves K, 1 moves V,
// 2 moves base and pos. Tiles of 64 slots are processed front to back; a tile is read completely
// into shared memory before any of it is written, and every destination index is <= its source
// index, so a write can only land on slots whose old contents were already read.
constexpr int kStableTile = 64;
__global__ void __launch_bounds__(256)
compact_stable_kernel(int Hkv, int cap, int row_bytes, char* __restrict__ K, char* __restrict__ V,
                      float* __restrict__ base, int* __restrict__ pos, const int* __restrict__ len,
                      const int* __restrict__ evict_idx, int max_evict, const int* __restrict__ n_evict) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  extern __shared__ __align__(16) char tile[];  // kStableTile * max(row_bytes, 8)
  const int unit = blockIdx.x, b = unit / Hkv, which = blockIdx.y;
  const int k = n_evict[b];
  if (k <= 0) return;
  const int n = len[b];
  const int* E = evict_idx + (size_t)unit * max_evict;
  char* arr = (which == 0) ? K : V;
  if (which == 2 && !base && !pos) return;
  const int rb = (which == 2) ? 8 : row_bytes;
  const int chunks_per_row = rb / ((which == 2) ? 8 : 16);
  for (int s0 = E[0]; s0 < n; s0 += kStableTile) {
    const int rows = min(kStableTile, n - s0);
    for (int idx = threadIdx.x; idx < rows * chunks_per_row; idx += blockDim.x) {
      const int r = idx / chunks_per_row, c = idx % chunks_per_row;
      const size_t slot = (size_t)unit * cap + s0 + r;
      if (which == 2) {
        float bv = base ? base[slot] : 0.f;
        int pv = pos ? pos[slot] : 0;
        *reinterpret_cast<float*>(tile + r * 8) = bv;
        *reinterpret_cast<int*>(tile + r * 8 + 4) = pv;
      } else {
        *reinterpret_cast<uint4*>(tile + (size_t)r * rb + c * 16) =
            *reinterpret_cast<const uint4*>(arr + slot * rb + c * 16);
      }
    }
    __syncthreads();
    for (int idx = threadIdx.x; idx < rows * chunks_per_row; idx += blockDim.x) {
      const int r = idx / chunks_per_row, c = idx % chunks_per_row;
      const int s = s0 + r;
      const int lb = lower_bound(E, k, s);
      if (lb < k && E[lb] == s) continue;  // evicted
      const size_t dst = (size_t)unit * cap + (s - lb);
      if (which == 2) {
        if (base) base[dst] = *reinterpret_cast<float*>(tile + r * 8);
        if (pos) pos[dst] = *reinterpret_cast<int*>(tile + r * 8 + 4);
      } else {
        *reinterpret_cast<uint4*>(arr + dst * rb + c * 16) =
            *reinterpret_cast<const uint4*>(tile + (size_t)r * rb + c * 16);
      }
    }
    __syncthreads();
  }
}

// len[b] -= n_evict[b], after every unit of the sequence has been compacted.
__global__ void update_len_kernel(int B, int* __restrict__ len, const int* __restrict__ n_evict) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < B) len[b] -= n_evict[b];
}

// Append m new rows per unit: grid = (units, ceil(m / 8)), 8 warps per CTA, one warp per row.
__global__ void __launch_bounds__(256)
append_kernel(int Hkv, int cap, int m, int row_bytes, char* __restrict__ K, char* __restrict__ V,
              float* __restrict__ base, int* __restrict__ pos, int* __restrict__ len,
              int* __restrict__ n_seen, const char* __restrict__ k_new,
              const char* __restrict__ v_new, int* status, int B, int* ticket) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  const int unit = blockIdx.x, b = unit / Hkv;
  const int n = len[b];
  const bool fits = n >= 0 && n + m <= cap;
  if (!fits && threadIdx.x == 0 && blockIdx.y == 0) set_status(status, CAOTE_ERR_OVERFLOW);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
  const int seen = n_seen ? n_seen[b] : n;
  for (int i = blockIdx.y * nwarps + warp; fits && i < m; i += gridDim.y * nwarps) {
    const size_t dst = (size_t)unit * cap + n + i, src = (size_t)unit * m + i;
    warp_copy_row(K + dst * row_bytes, k_new + src * row_bytes, row_bytes, lane);
    warp_copy_row(V + dst * row_bytes, v_new + src * row_bytes, row_bytes, lane);
    if (lane == 0) {
      if (base) base[dst] = 0.f;
      if (pos) pos[dst] = seen + i;
    }
  }
  // the CTA that finishes last moves the lengths on: len[b] += m and n_seen[b] += m for the
  // sequences that were not skipped (a ticket counter in the workspace header, reset here)
  __shared__ int s_last;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    s_last = (atomicAdd(ticket, 1) == (int)(gridDim.x * gridDim.y) - 1);
  }
  __syncthreads();
  if (s_last) {
    __threadfence();
    for (int bb = threadIdx.x; bb < B; bb += blockDim.x) {
      const int nb = len[bb];
      if (nb >= 0 && nb + m <= cap) {
        len[bb] = nb + m;
        if (n_seen) n_seen[bb] += m;
      }
    }
    if (threadIdx.x == 0) *ticket = 0;
  }
}

// Append of a few rows (Hkv * m <= 16): one CTA per sequence, a warp for each K row and each V row. The CTA reads the
// sequence's length once, so it can move it on itself after a barrier and no counter over the CTAs is needed.
// block = 64 * Hkv * m threads. With vsum (FastCAOTE, m = 1 only: one row per unit, so nobody else touches the unit's
// sums) the new value row is also added to the unit's running sum of value rows.
__global__ void __launch_bounds__(1024)
append_seq_kernel(int Hkv, int cap, int m, int row_bytes, char* __restrict__ K, char* __restrict__ V,
                  float* __restrict__ base, int* __restrict__ pos, int* __restrict__ len, int* __restrict__ n_seen,
                  const char* __restrict__ k_new, const char* __restrict__ v_new, int* status, float* __restrict__ vsum,
                  int elt_bytes) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n = len[b];
  const int seen = n_seen ? n_seen[b] : n;
  if (n < 0 || n + m > cap) {  // the sequence is skipped, its lengths stay
    if (threadIdx.x == 0) set_status(status, CAOTE_ERR_OVERFLOW);
    return;
  }
  const int r = warp >> 1, h = r / m, i = r % m;  // row r of the sequence: KV head h, new token i
  const int unit = b * Hkv + h;
  const size_t dst = (size_t)unit * cap + n + i, src = (size_t)unit * m + i;
  if (warp & 1) {
    if (vsum) {
      for (int o = lane * 16; o < row_bytes; o += 32 * 16) {
        const uint4 v = *reinterpret_cast<const uint4*>(v_new + src * row_bytes + o);
        *reinterpret_cast<uint4*>(V + dst * row_bytes + o) = v;
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        float* vs = vsum + (size_t)unit * (row_bytes / elt_bytes) + o / elt_bytes;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          if (elt_bytes == 2) {
            vs[2 * e] += __uint_as_float(w[e] << 16);
            vs[2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
          } else {
            vs[e] += __uint_as_float(w[e]);
          }
        }
      }
    } else {
      warp_copy_row(V + dst * row_bytes, v_new + src * row_bytes, row_bytes, lane);
    }
  } else {
    warp_copy_row(K + dst * row_bytes, k_new + src * row_bytes, row_bytes, lane);
    if (lane == 0) {
      if (base) base[dst] = 0.f;
      if (pos) pos[dst] = seen + i;
    }
  }
  __syncthreads();  // every warp has read the lengths
  if (threadIdx.x == 0) {
    len[b] = n + m;
    if (n_seen) n_seen[b] = seen + m;
  }
}

}  // namespace sel
}  // namespace caote
