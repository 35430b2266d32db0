// FastCAOTE (Sec. 3.3): the CAOTE score with X replaced by the plain mean of the cached values. The mean
// does not depend on this call's attention, so it can be carried from step to step: the library keeps
// vsum[u, :] = sum over the unit's valid slots of V[u, j, :] (fp32) and divides by n when it scores.
//   vsum_kernel        from scratch (one read of V)
//   vsum_add_kernel    += the m rows about to be appended
//   vsum_sub_unit      -= the rows about to be evicted (device function, used by the compaction kernels)
//   mean_kernel        X[u, :] = vsum[u, :] / n into the scratch location the score kernels read X from
#pragma once

#include "common.cuh"

namespace caote {
namespace fast {

// grid = units, 256 threads; D in {64, 128}.
template <typename T>
__global__ void __launch_bounds__(256)
vsum_kernel(int Hkv, int cap, int D, const T* __restrict__ V, const int* __restrict__ len, float* __restrict__ vsum) {
  __shared__ float part[256];
  const int unit = blockIdx.x, n = len[unit / Hkv];
  const int lanes = 256 / D, c = threadIdx.x % D, r0 = threadIdx.x / D;
  float acc = 0.f;
  if (n > 0 && n <= cap)
    for (int j = r0; j < n; j += lanes) acc += to_float(V[((size_t)unit * cap + j) * D + c]);
  part[threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.x < D) {
    float s = 0.f;
    for (int r = 0; r < lanes; ++r) s += part[r * D + threadIdx.x];
    vsum[(size_t)unit * D + threadIdx.x] = s;
  }
}

// grid = units, D threads. A sequence that caote_append will skip (no room for m rows) is skipped here too.
template <typename T>
__global__ void vsum_add_kernel(int Hkv, int cap, int m, int D, const T* __restrict__ v_new, const int* __restrict__ len,
                                float* __restrict__ vsum) {
  const int unit = blockIdx.x, n = len[unit / Hkv], c = threadIdx.x;
  if (n < 0 || n + m > cap) return;
  float acc = 0.f;
  for (int i = 0; i < m; ++i) acc += to_float(v_new[((size_t)unit * m + i) * D + c]);
  vsum[(size_t)unit * D + c] += acc;
}

// The rows listed in evict_idx[unit, 0..k) leave the sum; called by all threads of the unit's CTA before
// the rows are overwritten.
template <typename T>
__device__ inline void vsum_sub_unit(int unit, int k, int cap, int D, const T* __restrict__ V, const int* E,
                                     float* __restrict__ vsum) {  // (E: global or shared memory, possibly written by this CTA)
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    float acc = 0.f;
    for (int r = 0; r < k; ++r) acc += to_float(V[((size_t)unit * cap + E[r]) * D + c]);
    vsum[(size_t)unit * D + c] -= acc;
  }
}

// grid = units, 128 threads (the unfused selection / compaction path).
template <typename T>
__global__ void vsum_sub_kernel(int Hkv, int cap, int D, const T* __restrict__ V, const int* __restrict__ evict_idx,
                                int max_evict, const int* __restrict__ n_evict, float* __restrict__ vsum) {
  const int unit = blockIdx.x, k = n_evict[unit / Hkv];
  if (k > 0) vsum_sub_unit<T>(unit, k, cap, D, V, evict_idx + (size_t)unit * max_evict, vsum);
}

// grid = units, D threads.
__global__ void mean_kernel(int Hkv, int cap, int D, const int* __restrict__ len, const float* __restrict__ vsum,
                            float* __restrict__ X) {
  const int unit = blockIdx.x, n = len[unit / Hkv];
  if (n <= 0 || n > cap) return;
  X[(size_t)unit * D + threadIdx.x] = vsum[(size_t)unit * D + threadIdx.x] / (float)n;
}

}  // namespace fast
}  // namespace caote
