// Greedy multi-token eviction (Appendix B of the paper, the two-token derivation chained): evict the token
// whose removal changes the current output least, renormalise the weights of the rest, update the output,
// and score again, k times. One CTA per (sequence, KV head) unit.
//
// State kept on chip for the whole sequence of picks: the tokens' un-normalised weights h_j (negative once
// evicted) and the current distances in shared memory, the un-normalised output Y = sum_j h_j v_j and the
// normaliser H = sum_j h_j in registers / shared memory (X = Y / H). Every pick sweeps the unit's value rows
// once (a warp per token, its lanes over the channels, || X - v_j ||^2 by plain subtraction as on the
// scoring path): the rows come from HBM the first time and from L2 afterwards (a unit's rows are
// cap * d * element size, 1 MB at 4224 tokens). Per pick: that sweep, a block-wide arg-min over
// (score bits, position), and the rank-one update Y -= h_e v_e, H -= h_e.
#pragma once

#include "common.cuh"

namespace caote {
namespace greedy {

constexpr int kThreads = 1024;
constexpr int kWarps = kThreads / 32;
constexpr int kMaxTokens = 24576;  // two floats per token in shared memory

inline size_t smem_bytes(int cap, int D) {
  return sizeof(float) * ((size_t)2 * cap + 2 * D + 2 * kWarps) + sizeof(unsigned long long) * kWarps + sizeof(int) * kWarps + 64;
}

// CPL consecutive channels of a row as floats, with one vector load (the row pointer is 16-byte aligned, CPL = 2 or 4).
template <int CPL>
__device__ __forceinline__ void load_channels(const __nv_bfloat16* p, float (&f)[CPL]) {
  if constexpr (CPL == 4) {
    const uint2 r = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(r.x << 16); f[1] = __uint_as_float(r.x & 0xffff0000u);
    f[2] = __uint_as_float(r.y << 16); f[3] = __uint_as_float(r.y & 0xffff0000u);
  } else {
    const uint32_t r = *reinterpret_cast<const uint32_t*>(p);
    f[0] = __uint_as_float(r << 16); f[1] = __uint_as_float(r & 0xffff0000u);
  }
}
template <int CPL>
__device__ __forceinline__ void load_channels(const float* p, float (&f)[CPL]) {
  if constexpr (CPL == 4) {
    const float4 r = *reinterpret_cast<const float4*>(p);
    f[0] = r.x; f[1] = r.y; f[2] = r.z; f[3] = r.w;
  } else {
    const float2 r = *reinterpret_cast<const float2*>(p);
    f[0] = r.x; f[1] = r.y;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads, 1)
greedy_kernel(int Hkv, int cap, const T* __restrict__ V, const float* __restrict__ h_in, const int* __restrict__ len,
              const int* __restrict__ budget, const int* __restrict__ pos, int* __restrict__ evict_idx,
              int* __restrict__ order_out, int max_evict, int* __restrict__ n_evict, int* status) {
  constexpr int CPL = D / 32;  // channels per lane: lane l owns channels [l * CPL, (l + 1) * CPL)
  extern __shared__ __align__(16) float gsm[];
  float* hs = gsm;                   // [cap] weight of the token, < 0 once evicted
  float* ds = hs + cap;              // [cap] || X - v_j || of the current state
  float* Ys = ds + cap;              // [D]   sum of h_j v_j over the tokens present
  float* Ypart = Ys + D;             // [D]   scratch
  float* wsum = Ypart + D;           // [2 * kWarps]
  unsigned long long* wkey = reinterpret_cast<unsigned long long*>(wsum + 2 * kWarps);  // [kWarps]
  int* wslot = reinterpret_cast<int*>(wkey + kWarps);                                      // [kWarps]
  __shared__ float s_H;
  __shared__ int s_pick;

  const int unit = blockIdx.x, b = unit / Hkv, hd = unit % Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = len[b];
  int bud = budget[b];
  if (bud < 1) bud = 1;
  int k = n - bud;
  if (k < 0 || n > cap) k = 0;
  if (k > max_evict) {
    if (tid == 0) set_status(status, CAOTE_ERR_OVERFLOW);
    k = 0;
  }
  if (hd == 0 && tid == 0) n_evict[b] = k;
  if (k == 0) return;
  const T* Vu = V + (size_t)unit * cap * D;
  const float* hu = h_in + (size_t)unit * cap;
  const int* pu = pos ? pos + (size_t)unit * cap : nullptr;
  int* out = evict_idx + (size_t)unit * max_evict;
  int* ord = order_out ? order_out + (size_t)unit * max_evict : nullptr;

  // ---- H = sum h, Y = sum h v (one sweep; a warp per token, fixed order of the partial sums) ----
  float hsum = 0.f;
  for (int j = tid; j < n; j += kThreads) {
    const float hj = fmaxf(hu[j], 0.f);
    hs[j] = hj;
    hsum += hj;
  }
  hsum = warp_sum(hsum);
  if (lane == 0) wsum[warp] = hsum;
  float yacc[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) yacc[c] = 0.f;
  __syncthreads();
  for (int j = warp; j < n; j += kWarps) {
    const float hj = hs[j];
    float vf[CPL];
    load_channels<CPL>(Vu + (size_t)j * D + lane * CPL, vf);
#pragma unroll
    for (int c = 0; c < CPL; ++c) yacc[c] = fmaf(hj, vf[c], yacc[c]);
  }
  if (tid < D) Ys[tid] = 0.f;
  __syncthreads();
  for (int w = 0; w < kWarps; ++w) {  // warps add their parts one after the other: reproducible
    if (warp == w) {
#pragma unroll
      for (int c = 0; c < CPL; ++c) Ys[lane * CPL + c] += yacc[c];
    }
    __syncthreads();
  }
  if (tid == 0) {
    float H = 0.f;
    for (int w = 0; w < kWarps; ++w) H += wsum[w];
    s_H = H;
  }
  __syncthreads();

  for (int t = 0; t < k; ++t) {
    const float H = s_H;
    const float inv_H = (H > 0.f) ? 1.f / H : 0.f;
    // ---- distances of the tokens present to the current output: four rows per warp at a time, eight lanes per
    //      row, each with the 16-byte pieces l, l + 8, ... of the row (a row's loads are contiguous over its lanes) and
    //      three shuffle steps per sum; four such passes' loads in flight (a warp per row with a five-step sum kept
    //      the SM's one shuffle per clock busy for most of the sweep) ----
    {
      constexpr int E = 16 / (int)sizeof(T);  // elements per 16-byte piece
      constexpr int NCH = D / 8 / E;          // pieces per lane
      constexpr int kPasses = 8 / NCH;  // the passes in flight hold 32 registers of row pieces
      const int sub = lane >> 3, l8 = lane & 7;
      float x[NCH][E];
#pragma unroll
      for (int i = 0; i < NCH; ++i)
#pragma unroll
        for (int e = 0; e < E; ++e) x[i][e] = Ys[(l8 + 8 * i) * E + e] * inv_H;
      for (int j0 = 4 * warp; j0 < n; j0 += 4 * kWarps * kPasses) {
        uint4 raw[kPasses][NCH];
        bool live[kPasses];
#pragma unroll
        for (int u = 0; u < kPasses; ++u) {
          const int j = j0 + u * 4 * kWarps + sub;
          live[u] = j < n && hs[j] >= 0.f;
          if (live[u]) {
            const uint4* row = reinterpret_cast<const uint4*>(Vu + (size_t)j * D);
#pragma unroll
            for (int i = 0; i < NCH; ++i) raw[u][i] = row[l8 + 8 * i];
          }
        }
#pragma unroll
        for (int u = 0; u < kPasses; ++u) {
          float acc = 0.f;
          if (live[u]) {
#pragma unroll
            for (int i = 0; i < NCH; ++i) {
              const uint32_t w[4] = {raw[u][i].x, raw[u][i].y, raw[u][i].z, raw[u][i].w};
#pragma unroll
              for (int c = 0; c < 4; ++c) {
                if constexpr (sizeof(T) == 2) {
                  const float d0 = x[i][2 * c] - __uint_as_float(w[c] << 16);
                  const float d1 = x[i][2 * c + 1] - __uint_as_float(w[c] & 0xffff0000u);
                  acc = fmaf(d0, d0, fmaf(d1, d1, acc));
                } else {
                  const float d0 = x[i][c] - __uint_as_float(w[c]);
                  acc = fmaf(d0, d0, acc);
                }
              }
            }
          }
          acc += __shfl_xor_sync(0xffffffffu, acc, 4);
          acc += __shfl_xor_sync(0xffffffffu, acc, 2);
          acc += __shfl_xor_sync(0xffffffffu, acc, 1);
          if (live[u] && l8 == 0) ds[j0 + u * 4 * kWarps + sub] = sqrtf(acc);
        }
      }
    }
    __syncthreads();
    // ---- arg-min of w_j / (1 - w_j) * dist_j over (score bits, position) ----
    unsigned long long best = ~0ull;
    int best_slot = -1;
    for (int j = tid; j < n; j += kThreads) {
      const float hj = hs[j];
      if (hj < 0.f) continue;
      float sc = 0.f;
      if (H > 0.f && hj > 0.f) {
        const float rest = H - hj;  // the others' weight (times H)
        sc = (rest > 0.f) ? hj / rest * ds[j] : INFINITY;
      }
      const unsigned long long key = ((unsigned long long)__float_as_uint(sc) << 32) | (unsigned int)(pu ? pu[j] : j);
      if (key < best) { best = key; best_slot = j; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok = __shfl_xor_sync(0xffffffffu, best, o);
      const int os = __shfl_xor_sync(0xffffffffu, best_slot, o);
      if (ok < best) { best = ok; best_slot = os; }
    }
    if (lane == 0) { wkey[warp] = best; wslot[warp] = best_slot; }
    __syncthreads();
    if (tid == 0) {
      unsigned long long bk = wkey[0];
      int bs = wslot[0];
      for (int w = 1; w < kWarps; ++w)
        if (wkey[w] < bk) { bk = wkey[w]; bs = wslot[w]; }
      s_pick = bs;
    }
    __syncthreads();
    const int e = s_pick;
    if (e < 0) break;  // (cannot happen with k < n; keeps every index in bounds)
    // ---- evict e: Y -= h_e v_e, H -= h_e ----
    const float he = hs[e];
    if (tid < D) Ys[tid] -= he * to_float(Vu[(size_t)e * D + tid]);
    if (tid == 0) {
      s_H = H - he;
      if (ord) ord[t] = e;
    }
    __syncthreads();
    if (tid == 0) hs[e] = -1.f;
    __syncthreads();
  }
  // ---- the evicted slots in ascending order (the layout caote_compact expects) ----
  __shared__ int s_count;
  if (tid == 0) s_count = 0;
  __syncthreads();
  for (int j0 = 0; j0 < n; j0 += kThreads) {
    const int j = j0 + tid;
    const bool gone = j < n && hs[j] < 0.f;
    const unsigned m = __ballot_sync(0xffffffffu, gone);
    if (lane == 0) wslot[warp] = __popc(m);
    __syncthreads();
    int before = s_count;
    for (int w = 0; w < warp; ++w) before += wslot[w];
    if (gone) out[before + __popc(m & ((1u << lane) - 1u))] = j;
    __syncthreads();
    if (tid == 0) {
      int tot = s_count;
      for (int w = 0; w < kWarps; ++w) tot += wslot[w];
      s_count = tot;
    }
    __syncthreads();
  }
}

}  // namespace greedy
}  // namespace caote
