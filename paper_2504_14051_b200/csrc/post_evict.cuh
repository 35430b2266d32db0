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
// Blocks of queries with per-row statistics (the tensor-core prefill kernels) have a kernel of their own further
// down, which shares the evicted rows among 32 query rows; this one then leaves those calls alone.
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
                  const int* __restrict__ stat_tag, const float* __restrict__ stats, int prefill_stride,
                  int rows_kernel_ran) {
  constexpr int LD = D + 4, CPL = D / 32;  // channels per lane
  if (rows_kernel_ran && stat_tag && *stat_tag == kStatPerRow) return;  // post_evict_rows_kernel has done the work
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
    stat2 = (tag == kStatPerHead) ? stats[(size_t)unit * kHeadStatFloats + g] : stats[(size_t)unit * prefill_stride + r];
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

// The same correction for blocks of queries whose rows' statistics the scoring call left behind (bf16, head_dim 128):
// does nothing unless the workspace header says so. A CTA takes 16 query rows of a unit (two per warp) and walks
// the unit's evicted slots 32 at a time: their K and V rows are gathered into shared memory once for all its query
// rows; for the logits a lane is an evicted token (its K row against the warp's four query rows, both from shared
// memory), for the weighted value sum a lane is four channels. grid = (ceil(R / 16), units), 256 threads.
constexpr int kRowsPerWarp = 2, kBlockRows = 8 * kRowsPerWarp, kChunk = 32, kRowsD = 128, kKLd = kRowsD + 1;
inline size_t rows_smem_bytes() {
  return sizeof(float) * ((size_t)kBlockRows * kRowsD + (size_t)kChunk * kKLd + (size_t)kChunk * kRowsD + (size_t)kBlockRows * kChunk) +
         sizeof(int) * kChunk;
}

__global__ void __launch_bounds__(256)
post_evict_rows_kernel(Dims dm, const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ K,
                       const __nv_bfloat16* __restrict__ V, const int* __restrict__ len,
                       const int* __restrict__ evict_idx, int max_evict, const int* __restrict__ n_evict,
                       const float* __restrict__ o, float* __restrict__ o_post, const int* __restrict__ stat_tag,
                       const float* __restrict__ stats, int stat_stride) {
  constexpr int D = kRowsD;
  if (*stat_tag != kStatPerRow) return;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;                        // [kBlockRows][D]
  float* Ks = Qs + kBlockRows * D;         // [kChunk][kKLd]   (odd row pitch: a lane per row, no bank conflicts)
  float* Vs = Ks + kChunk * kKLd;          // [kChunk][D]
  float* As = Vs + kChunk * D;             // [kBlockRows][kChunk] weights of the chunk
  int* js = reinterpret_cast<int*>(As + kBlockRows * kChunk);  // [kChunk] slot of the evicted token, -1: none
  const int unit = blockIdx.y, b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b], m = dm.m;
  if (n <= 0 || n < m || n > dm.cap) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r0 = blockIdx.x * kBlockRows;
  const float scale2 = dm.scale * 1.4426950408889634f;
  auto row_off = [&](int r) { return (((size_t)b * dm.Hq + h * dm.G + r / m) * m + r % m) * D; };
  for (int idx = tid; idx < kBlockRows * D; idx += 256) {
    const int rr = idx / D, c = idx % D, r = r0 + rr;
    Qs[idx] = (r < dm.R) ? __bfloat162float(q[row_off(r) + c]) : 0.f;
  }
  constexpr int RW = kRowsPerWarp;
  int n_vis[RW];
  float stat[RW], A[RW], Y[RW][4];
#pragma unroll
  for (int i = 0; i < RW; ++i) {
    const int r = r0 + RW * warp + i;
    n_vis[i] = (r < dm.R) ? n - m + (r % m) + 1 : 0;
    stat[i] = (r < dm.R) ? stats[(size_t)unit * stat_stride + r] : 0.f;
    A[i] = 0.f;
#pragma unroll
    for (int c = 0; c < 4; ++c) Y[i][c] = 0.f;
  }
  const int k = n_evict[b];
  const int* E = evict_idx + (size_t)unit * max_evict;
  const __nv_bfloat16* Ku = K + (size_t)unit * dm.cap * D;
  const __nv_bfloat16* Vu = V + (size_t)unit * dm.cap * D;
  for (int e0 = 0; e0 < k; e0 += kChunk) {
    __syncthreads();  // (the query rows are staged; the previous chunk is used up)
    // gather: warp w brings tokens 4 w .. 4 w + 3 of the chunk, a lane four channels of a row
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int tok = 4 * warp + t, e = e0 + tok;
      int j = (e < k) ? E[e] : -1;
      if (j < 0 || j >= n) j = -1;
      float kf[4] = {0.f, 0.f, 0.f, 0.f}, vf[4] = {0.f, 0.f, 0.f, 0.f};
      if (j >= 0) {
        const uint2 kr = *reinterpret_cast<const uint2*>(Ku + (size_t)j * D + 4 * lane);
        const uint2 vr = *reinterpret_cast<const uint2*>(Vu + (size_t)j * D + 4 * lane);
        kf[0] = __uint_as_float(kr.x << 16); kf[1] = __uint_as_float(kr.x & 0xffff0000u);
        kf[2] = __uint_as_float(kr.y << 16); kf[3] = __uint_as_float(kr.y & 0xffff0000u);
        vf[0] = __uint_as_float(vr.x << 16); vf[1] = __uint_as_float(vr.x & 0xffff0000u);
        vf[2] = __uint_as_float(vr.y << 16); vf[3] = __uint_as_float(vr.y & 0xffff0000u);
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) Ks[tok * kKLd + 4 * lane + c] = kf[c];
      *reinterpret_cast<float4*>(Vs + tok * D + 4 * lane) = make_float4(vf[0], vf[1], vf[2], vf[3]);
      if (lane == 0) js[tok] = j;
    }
    __syncthreads();
    // weights: lane = evicted token of the chunk
    {
      const int j = js[lane];
      float s[RW];
#pragma unroll
      for (int i = 0; i < RW; ++i) s[i] = 0.f;
      const float* kp = Ks + lane * kKLd;
#pragma unroll 8
      for (int c = 0; c < D; c += 4) {
        const float k0 = kp[c], k1 = kp[c + 1], k2 = kp[c + 2], k3 = kp[c + 3];
#pragma unroll
        for (int i = 0; i < RW; ++i) {
          const float4 q4 = *reinterpret_cast<const float4*>(Qs + (RW * warp + i) * D + c);
          s[i] = fmaf(q4.x, k0, fmaf(q4.y, k1, fmaf(q4.z, k2, fmaf(q4.w, k3, s[i]))));
        }
      }
#pragma unroll
      for (int i = 0; i < RW; ++i) {
        const float a = (j >= 0 && j < n_vis[i]) ? exp2f(fmaf(s[i], scale2, -stat[i])) : 0.f;
        A[i] += a;
        As[(RW * warp + i) * kChunk + lane] = a;
      }
    }
    __syncwarp();  // (a warp reads only the weights it wrote)
    // weighted values: lane = four channels
#pragma unroll 4
    for (int t = 0; t < kChunk; ++t) {
      const float4 v4 = *reinterpret_cast<const float4*>(Vs + t * D + 4 * lane);
#pragma unroll
      for (int i = 0; i < RW; ++i) {
        const float a = As[(RW * warp + i) * kChunk + t];
        Y[i][0] = fmaf(a, v4.x, Y[i][0]);
        Y[i][1] = fmaf(a, v4.y, Y[i][1]);
        Y[i][2] = fmaf(a, v4.z, Y[i][2]);
        Y[i][3] = fmaf(a, v4.w, Y[i][3]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < RW; ++i) {
    const int r = r0 + RW * warp + i;
    const float rest = 1.f - warp_sum(A[i]);
    if (r < dm.R) {
      const size_t at = row_off(r) + 4 * lane;
      const float4 o4 = *reinterpret_cast<const float4*>(o + at);
      float4 res = make_float4(0.f, 0.f, 0.f, 0.f);
      if (rest > 0.f) res = make_float4((o4.x - Y[i][0]) / rest, (o4.y - Y[i][1]) / rest, (o4.z - Y[i][2]) / rest, (o4.w - Y[i][3]) / rest);
      *reinterpret_cast<float4*>(o_post + at) = res;
    }
  }
}

}  // namespace post
}  // namespace caote
