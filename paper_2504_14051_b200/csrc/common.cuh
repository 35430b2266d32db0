// Shared device/host helpers of the CAOTE CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/caote.h"

namespace caote {

// ---- workspace layout -------------------------------------------------------------------------
// [0, 256)            header: int32 status word at offset 0
// [256, ...)          per-call scratch, carved by the entry point that uses it
constexpr size_t kHeaderBytes = 256;
// Word kStatTagIndex of the workspace header says which softmax statistics the last scoring call left at
// workspace + kHeaderBytes for the post-eviction output to reuse (reference + log2(sum) of the log2-domain
// logits): per query head of a unit ([units][kHeadStatFloats], single-query kernels), per query row of a unit
// ([units][padded rows], tensor-core prefill kernels), or none.
constexpr int kStatTagIndex = 8;
constexpr int kStatNone = 0, kStatPerHead = 1, kStatPerRow = 2;
// Per query head the record is three rows of 8 floats per unit: the log-sum-exp, the largest logit, and the share of
// all the other tokens next to the token that holds it (sum of the others / sum); the last two only from the
// cluster kernel, for the sum-of-errors pass that follows it.
constexpr int kHeadStatFloats = 24;

struct Dims {
  int B, Hq, Hkv, G, D, cap, m, R;  // R = G * m query rows per unit
  int units;                         // B * Hkv
  float scale;
  int base_mode;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// SMs of the current device, as far as the host-side split heuristics are concerned. The entry points refresh
// it from the device attribute before they size or carve a workspace; without a device it stays at 148.
inline int g_sm_count = 148;

// Record the first device-side error in the status word (never overwrites an earlier one).
__device__ inline void set_status(int* status, int code) { atomicCAS(status, 0, code); }

// ---- element access ---------------------------------------------------------------------------
__device__ inline float to_float(float x) { return x; }
__device__ inline float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ inline T from_float(float x);
template <>
__device__ inline float from_float<float>(float x) { return x; }
template <>
__device__ inline __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load 4 consecutive elements (16-byte aligned for float, 8-byte for bf16) as floats.
__device__ inline float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ inline float4 load4(const __nv_bfloat16* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  const float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}

// Load 8 consecutive bf16 (16-byte aligned) as floats.
__device__ inline void load8(const __nv_bfloat16* p, float* out) {
  const uint4 raw = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    out[2 * i] = f.x;
    out[2 * i + 1] = f.y;
  }
}

__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

}  // namespace caote
