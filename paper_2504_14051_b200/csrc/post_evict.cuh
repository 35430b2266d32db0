// Post-eviction attention output (Sec. 2, budgeted generation; Sec. 3.1, proof of Theorem 3.2): what the
// output of each query row becomes once the evicted tokens are gone and the remaining attention weights
// are renormalised,
//     o'_r = (o_r - sum_{e in E} alpha_{r,e} v_e) / (1 - sum_{e in E} alpha_{r,e}),
// E = the evicted slots the row can see. The weights alpha_{r,e} need the row's softmax normaliser. Where the
// scoring call that ran just before on the same workspace has left the rows' statistics there (the cluster
// decode kernel: one per query head; the tensor-core prefill kernels: one per row; both as reference +
// log2(sum) of the log2-domain logits), they are used and the kernel touches only q, the evicted K / V rows
// and o; the kind of statistics present is a tag in the workspace header. Otherwise the normaliser is
// recomputed with one pass over K (fp32 on the CUDA cores, any dtype, head_dim 64 or 128).
// grid = (ceil(R / kRows), units), 256 threads: one warp per query row.
#pragma once

#include "common.cuh"

namespace caote {
namespace post {

constexpr int kRows = 8;
constexpr int kKeys = 64;

template <int D>
inline size_t smem_bytes() { return sizeof(float) * ((size_t)kKeys * (D + 4) + (size_t)kRows * D); }

template <typename T, int D>
__global__ void __launch_bounds__(32 * kRows)
post_evict_kernel(Dims dm, const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                  const int* __restrict__ len, const int* __restrict__ evict_idx, int max_evict,
                  const int* __restrict__ n_evict, const float* __restrict__ o, float* __restrict__ o_post,
                  const int* __restrict__ stat_tag, const float* __restrict__ stats, int prefill_stride) {
  constexpr int LD = D + 4, CPL = D / 32;  // channels per lane
  extern __shared__ __align__(16) float smem[];
  float* Ks = smem;             // [kKeys][LD]
  float* Qs = Ks + kKeys * LD;  // [kRows][D]
  const int unit = blockIdx.y, b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b], m = dm.m;
  if (n <= 0 || n < m || n > dm.cap) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = blockIdx.x * kRows + warp;
  const bool row_ok = r < dm.R;
  const int g = row_ok ? r / m : 0, i = row_ok ? r % m : 0;
  const size_t qoff = (((size_t)b * dm.Hq + h * dm.G + g) * m + i) * D;
  const int n_vis = row_ok ? n - m + i + 1 : 0;
  for (int c = lane; c < D; c += 32) Qs[warp * D + c] = row_ok ? to_float(q[qoff + c]) : 0.f;
  const T* Ku = K + (size_t)unit * dm.cap * D;
  const T* Vu = V + (size_t)unit * dm.cap * D;

  // statistics left by the scoring call? (1: per query head, 2: per row; anything else: none)
  const int tag = stat_tag ? *stat_tag : 0;
  const bool have_stat = (tag == kStatPerHead && m == 1) || tag == kStatPerRow;
  float stat2 = 0.f;  // alpha = 2^(log2(e) * scale * <q, k> - stat2)
  if (have_stat && row_ok)
    stat2 = (tag == kStatPerHead) ? stats[(size_t)unit * 8 + g] : stats[(size_t)unit * prefill_stride + r];
  // pass over the keys: running maximum and sum of exp of this row's logits, two keys per lane and tile
  float mx = -INFINITY, l = 0.f;
  for (int kt = 0; kt < (have_stat ? 0 : n); kt += kKeys) {
    __syncthreads();
    for (int idx = tid; idx < kKeys * (D / 4); idx += blockDim.x) {
      const int rr = idx / (D / 4), c4 = idx % (D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (kt + rr < n) v = load4(Ku + (size_t)(kt + rr) * D + c4 * 4);
      *reinterpret_cast<float4*>(Ks + rr * LD + c4 * 4) = v;
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int jj = lane + 32 * t, j = kt + jj;
      if (j < n_vis) {
        float s = 0.f;
#pragma unroll 8
        for (int c = 0; c < D; c += 4) {
          const float4 kv = *reinterpret_cast<const float4*>(Ks + jj * LD + c);
          const float4 qv = *reinterpret_cast<const float4*>(Qs + warp * D + c);
          s = fmaf(qv.x, kv.x, s); s = fmaf(qv.y, kv.y, s); s = fmaf(qv.z, kv.z, s); s = fmaf(qv.w, kv.w, s);
        }
        s *= dm.scale;
        const float nm = fmaxf(mx, s);
        l = l * __expf(mx - nm) + __expf(s - nm);
        mx = nm;
      }
    }
  }
  const float M = warp_max(mx);
  const float Z = warp_sum(mx == -INFINITY ? 0.f : l * __expf(mx - M));
  if (!row_ok) return;

  // the evicted slots this row sees: their weights and weighted values (lane = CPL channels)
  const int k = n_evict[b];
  const int* E = evict_idx + (size_t)unit * max_evict;
  float A = 0.f, Y[CPL];
#pragma unroll
  for (int c = 0; c < CPL; ++c) Y[c] = 0.f;
  for (int e = 0; e < k; ++e) {
    const int j = E[e];
    if (j < 0 || j >= n_vis) continue;
    float part = 0.f, vv[CPL];
#pragma unroll
    for (int c = 0; c < CPL; ++c) {
      part = fmaf(Qs[warp * D + lane * CPL + c], to_float(Ku[(size_t)j * D + lane * CPL + c]), part);
      vv[c] = to_float(Vu[(size_t)j * D + lane * CPL + c]);
    }
    const float s = warp_sum(part) * dm.scale;
    const float a = have_stat ? exp2f(s * 1.4426950408889634f - stat2) : __expf(s - M) / Z;
    A += a;
#pragma unroll
    for (int c = 0; c < CPL; ++c) Y[c] = fmaf(a, vv[c], Y[c]);
  }
  const float rest = 1.f - A;
#pragma unroll
  for (int c = 0; c < CPL; ++c) {
    const size_t at = qoff + lane * CPL + c;
    o_post[at] = rest > 0.f ? (o[at] - Y[c]) / rest : 0.f;
  }
}

}  // namespace post
}  // namespace caote
