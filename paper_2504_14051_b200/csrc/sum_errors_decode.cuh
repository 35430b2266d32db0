// Sum-of-errors aggregation for a single query per head (bf16, head_dim 128, up to 8 query heads per KV head): the
// score of a cached token is the sum over the group's heads of the exact single-head eviction error (Sec. 3.1,
// Theorem 3.2),
//     c_j = sum_g alpha_{g,j} / (1 - alpha_{g,j}) * || o_g - v_j ||_2 .
// It runs after the cluster kernel, which has written the heads' outputs o_g and left per head the log-sum-exp m_g
// (alpha_{g,j} = 2^(s_{g,j} - m_g)), the largest logit and the share of all other tokens next to the token that
// holds it. This pass reads K and V once more: a CTA takes 128 tokens of a unit, their K and V rows land in shared
// memory by TMA (two boxes of 64 channels each, 128-byte swizzle), two threads share a token, each with half of the
// heads, and form their logits and distances by plain subtraction (no ||o||^2 - 2 o.v + ||v||^2: for a token that holds nearly all of a head's
// weight o_g is nearly v_j, and a bf16 cross term from the tensor cores would leave nothing of the difference).
// 1 - alpha of a head's top token is the stored share of the others, never a difference of nearly equal numbers.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace caote {
namespace sed {

constexpr int kT = 128;                      // tokens per CTA
constexpr int kThreads = 2 * kT;             // two threads per token: the heads are split between them
constexpr int kD = 128;
constexpr int kTileBytes = kT * kD * 2;      // a K or V tile
constexpr long long kWaitCycles = 2000000000LL;

inline size_t smem_bytes() { return 1024 + 2 * (size_t)kTileBytes + sizeof(float) * (2 * 8 * kD + 24 + kT) + 64; }

template <int G>
__global__ void __launch_bounds__(kThreads)
sum_errors_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, Dims dm,
                         const __nv_bfloat16* __restrict__ q, const int* __restrict__ len, const float* __restrict__ o,
                         const float* __restrict__ head_stats, float* __restrict__ scores, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  extern __shared__ char smem_raw[];
  char* sm = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  char* Ks = sm;
  char* Vs = Ks + kTileBytes;
  float* Qs = reinterpret_cast<float*>(Vs + kTileBytes);  // [8][kD]
  float* Os = Qs + 8 * kD;                                  // [8][kD]
  float* St = Os + 8 * kD;                                  // [3][8]
  float* Cx = St + 24;                                      // [kT] the second thread's part of a token's score
  uint64_t* bar = reinterpret_cast<uint64_t*>(Cx + kT);

  const int unit = blockIdx.y, b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b], j0 = blockIdx.x * kT;
  if (n <= 0 || n > dm.cap || j0 >= n) return;
  const int tid = threadIdx.x;
  if (tid == 0) {
    ptx::mbar_init(bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    ptx::mbar_expect_tx(bar, 2 * kTileBytes);
    const int row = unit * dm.cap + j0;
    ptx::tma_load_2d(Ks, &tmK, 0, row, bar);
    ptx::tma_load_2d(Ks + kTileBytes / 2, &tmK, 64, row, bar);
    ptx::tma_load_2d(Vs, &tmV, 0, row, bar);
    ptx::tma_load_2d(Vs + kTileBytes / 2, &tmV, 64, row, bar);
  }
  // the heads' queries, outputs and statistics
  const size_t qo = ((size_t)b * dm.Hq + (size_t)h * G) * kD;
  for (int i = tid; i < G * kD; i += kThreads) {
    Qs[i] = __bfloat162float(q[qo + i]);
    Os[i] = o[qo + i];
  }
  if (tid < 24) St[tid] = head_stats[(size_t)unit * kHeadStatFloats + tid];
  __syncthreads();
  if (!ptx::mbar_try_wait(bar, 0)) {
    const long long t0 = clock64();
    while (!ptx::mbar_try_wait(bar, 0)) {
      if (clock64() - t0 > kWaitCycles) {  // (the copy never came: say so and leave the scores alone)
        if (tid == 0) set_status(status, CAOTE_ERR_TIMEOUT);
        return;
      }
    }
  }
  // thread tok takes heads [0, GH), thread tok + 128 heads [GH, G)
  constexpr int GH = (G + 1) / 2;
  const int tok = tid & (kT - 1), g0 = (tid >> 7) * GH;
  const int j = j0 + tok;
  float s[GH], d2[GH];
#pragma unroll
  for (int g = 0; g < GH; ++g) { s[g] = 0.f; d2[g] = 0.f; }
  const float* Qh = Qs + g0 * kD;
  const float* Oh = Os + g0 * kD;
#pragma unroll 2
  for (int c = 0; c < 16; ++c) {  // 16 chunks of 8 channels
    const uint4 kr = *reinterpret_cast<const uint4*>(Ks + ptx::tile_off(tok, c));
    const uint4 vr = *reinterpret_cast<const uint4*>(Vs + ptx::tile_off(tok, c));
    const uint32_t kw[4] = {kr.x, kr.y, kr.z, kr.w}, vw[4] = {vr.x, vr.y, vr.z, vr.w};
    float kf[8], vf[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      kf[2 * e] = __uint_as_float(kw[e] << 16);
      kf[2 * e + 1] = __uint_as_float(kw[e] & 0xffff0000u);
      vf[2 * e] = __uint_as_float(vw[e] << 16);
      vf[2 * e + 1] = __uint_as_float(vw[e] & 0xffff0000u);
    }
#pragma unroll
    for (int g = 0; g < GH; ++g) {  // (a head index beyond G reads rows of the tables that exist and is dropped below)
      const float4 q0 = *reinterpret_cast<const float4*>(Qh + g * kD + 8 * c), q1 = *reinterpret_cast<const float4*>(Qh + g * kD + 8 * c + 4);
      const float4 o0 = *reinterpret_cast<const float4*>(Oh + g * kD + 8 * c), o1 = *reinterpret_cast<const float4*>(Oh + g * kD + 8 * c + 4);
      const float qq[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
      const float oo[8] = {o0.x, o0.y, o0.z, o0.w, o1.x, o1.y, o1.z, o1.w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        s[g] = fmaf(qq[e], kf[e], s[g]);
        const float df = oo[e] - vf[e];
        d2[g] = fmaf(df, df, d2[g]);
      }
    }
  }
  const float scale2 = dm.scale * 1.4426950408889634f;
  float cj = 0.f;
#pragma unroll
  for (int g = 0; g < GH; ++g) {
    if (g0 + g >= G) continue;
    const float s2 = s[g] * scale2;
    const float a = exp2f(s2 - St[g0 + g]);
    // the head's top token (its logit, formed here in another order than in the attention pass, within 3e-4 of the
    // largest): the others' share as stored; two tokens that close to the top have weights that close to each other
    const float rest = (s2 >= St[8 + g0 + g] - 3e-4f) ? St[16 + g0 + g] : 1.f - a;
    cj += (a == 0.f) ? 0.f : ((rest > 0.f) ? a / rest * sqrtf(d2[g]) : INFINITY);
  }
  if (tid >= kT) Cx[tok] = cj;
  __syncthreads();
  if (tid < kT && j < n) scores[(size_t)unit * dm.cap + j] = cj + Cx[tok];
}

}  // namespace sed
}  // namespace caote
