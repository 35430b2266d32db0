// Sum-of-errors aggregation for a single query per head (bf16, head_dim 128, up to 8 query heads per KV head): the
// score of a cached token is the sum over the group's heads of the exact single-head eviction error (Sec. 3.1,
// Theorem 3.2),
//     c_j = sum_g alpha_{g,j} / (1 - alpha_{g,j}) * || o_g - v_j ||_2 .
// It runs after the cluster kernel, which has written the heads' outputs o_g and left per head the log-sum-exp m_g
// (alpha_{g,j} = 2^(s_{g,j} - m_g)), the largest logit and the share of all other tokens next to the token that
// holds it. This pass reads K and V once more: a CTA takes 128 tokens of a unit, their K and V rows land in shared
// memory by TMA (two boxes of 64 channels each, 128-byte swizzle), a thread takes four tokens and a quarter of the
// heads (what bounds the pass on chip is the bytes that shared memory delivers to registers: the heads' q and o rows
// are fetched once per four tokens, 4 KB per token in all where two threads per token with half of the heads each
// took 9 KB), and forms logits and distances by plain subtraction (no ||o||^2 - 2 o.v + ||v||^2: for a token that holds nearly all of a head's
// weight o_g is nearly v_j, and a bf16 cross term from the tensor cores would leave nothing of the difference).
// 1 - alpha of a head's top token is the stored share of the others, never a difference of nearly equal numbers.
#pragma once

#include "common.cuh"
#include "ptx.cuh"

namespace caote {
namespace sed {

constexpr int kT = 128;                      // tokens per CTA
constexpr int kTok = 4;                      // tokens per thread: tq, tq + 32, tq + 64, tq + 96
constexpr int kThreads = 4 * (kT / kTok);    // warp w takes the w-th quarter of the heads
constexpr int kD = 128;
constexpr int kTileBytes = kT * kD * 2;      // a K or V tile
constexpr long long kWaitCycles = 2000000000LL;

inline size_t smem_bytes() { return 1024 + 2 * (size_t)kTileBytes + sizeof(float) * (2 * 8 * kD + 24 + 3 * kT) + 64; }

template <int G>
__global__ void __launch_bounds__(kThreads)
sum_errors_decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, Dims dm,
                         const __nv_bfloat16* __restrict__ q, const int* __restrict__ len, const float* __restrict__ o,
                         const float* __restrict__ head_stats, float* __restrict__ scores, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  extern __shared__ char smem_raw[];
  // (1024-byte alignment by an offset into the array, not by a round trip through an integer: the pointer keeps its
  // address space, so what is read through it compiles to shared-memory loads, not generic ones)
  char* sm = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  char* Ks = sm;
  char* Vs = Ks + kTileBytes;
  float* Qs = reinterpret_cast<float*>(Vs + kTileBytes);  // [8][kD]
  float* Os = Qs + 8 * kD;                                  // [8][kD], the heads' outputs negated
  float* St = Os + 8 * kD;                                  // [3][8]
  float* Cx = St + 24;                                      // [3][kT] the other head quarters' parts of a token's score
  uint64_t* bar = reinterpret_cast<uint64_t*>(Cx + 3 * kT);

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
    Os[i] = -o[qo + i];  // (negated: the distance pass forms v - o with a packed add)
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
  // lane tq of warp w: tokens tq + 32 t, heads [w GQ, (w + 1) GQ)
  constexpr int GQ = (G + 3) / 4;
  const int tq = tid & 31, g0 = (tid >> 5) * GQ;
  // logits and squared distances as pairs of partial sums over the even and the odd channels (packed fp32 math)
  float2 s[kTok][GQ], d2[kTok][GQ];
#pragma unroll
  for (int t = 0; t < kTok; ++t)
#pragma unroll
    for (int g = 0; g < GQ; ++g) { s[t][g] = make_float2(0.f, 0.f); d2[t][g] = make_float2(0.f, 0.f); }
  // (a head index beyond G reads rows of the tables that exist, 4 GQ <= 8, and is dropped below)
  const float* Qh = Qs + g0 * kD;
  const float* Oh = Os + g0 * kD;
#pragma unroll 1
  for (int c = 0; c < 16; ++c) {  // 16 chunks of 8 channels
    float2 qq[GQ][4], no[GQ][4];
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      const float4 q0 = *reinterpret_cast<const float4*>(Qh + g * kD + 8 * c), q1 = *reinterpret_cast<const float4*>(Qh + g * kD + 8 * c + 4);
      const float4 o0 = *reinterpret_cast<const float4*>(Oh + g * kD + 8 * c), o1 = *reinterpret_cast<const float4*>(Oh + g * kD + 8 * c + 4);
      qq[g][0] = make_float2(q0.x, q0.y); qq[g][1] = make_float2(q0.z, q0.w); qq[g][2] = make_float2(q1.x, q1.y); qq[g][3] = make_float2(q1.z, q1.w);
      no[g][0] = make_float2(o0.x, o0.y); no[g][1] = make_float2(o0.z, o0.w); no[g][2] = make_float2(o1.x, o1.y); no[g][3] = make_float2(o1.z, o1.w);
    }
#pragma unroll
    for (int t = 0; t < kTok; ++t) {
      const int tok = tq + 32 * t;
      const uint4 kr = *reinterpret_cast<const uint4*>(Ks + ptx::tile_off(tok, c));
      const uint4 vr = *reinterpret_cast<const uint4*>(Vs + ptx::tile_off(tok, c));
      const uint32_t kw[4] = {kr.x, kr.y, kr.z, kr.w}, vw[4] = {vr.x, vr.y, vr.z, vr.w};
      float2 kf[4], vf[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        kf[e] = make_float2(__uint_as_float(kw[e] << 16), __uint_as_float(kw[e] & 0xffff0000u));
        vf[e] = make_float2(__uint_as_float(vw[e] << 16), __uint_as_float(vw[e] & 0xffff0000u));
      }
#pragma unroll
      for (int g = 0; g < GQ; ++g) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          s[t][g] = __ffma2_rn(qq[g][e], kf[e], s[t][g]);
          const float2 df = __fadd2_rn(vf[e], no[g][e]);
          d2[t][g] = __ffma2_rn(df, df, d2[t][g]);
        }
      }
    }
  }
  const float scale2 = dm.scale * 1.4426950408889634f;
  float cj[kTok];
#pragma unroll
  for (int t = 0; t < kTok; ++t) {
    cj[t] = 0.f;
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      if (g0 + g >= G) continue;
      const float s2 = (s[t][g].x + s[t][g].y) * scale2;
      const float a = exp2f(s2 - St[g0 + g]);
      // the head's top token (its logit, formed here in another order than in the attention pass, within 3e-4 of the
      // largest): the others' share as stored; two tokens that close to the top have weights that close to each other
      const float rest = (s2 >= St[8 + g0 + g] - 3e-4f) ? St[16 + g0 + g] : 1.f - a;
      cj[t] += (a == 0.f) ? 0.f : ((rest > 0.f) ? a / rest * sqrtf(d2[t][g].x + d2[t][g].y) : INFINITY);
    }
    if (tid >= 32) Cx[((tid >> 5) - 1) * kT + tq + 32 * t] = cj[t];
  }
  __syncthreads();
  if (tid < 32) {
#pragma unroll
    for (int t = 0; t < kTok; ++t) {
      const int tok = tq + 32 * t, j = j0 + tok;
      if (j < n) scores[(size_t)unit * dm.cap + j] = cj[t] + Cx[tok] + Cx[kT + tok] + Cx[2 * kT + tok];
    }
  }
}

}  // namespace sed
}  // namespace caote
