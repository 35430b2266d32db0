// Single-query (decode) scoring path for bf16, head_dim 128, group size <= 8: one persistent kernel
// that reads K and V from HBM exactly once.
//
// Work is cut into chunks of kT consecutive cached tokens of one (sequence, KV head) unit; chunk c is
// handled by CTA c mod gridDim.x (one CTA per SM, all co-resident). For every chunk a CTA
//   1. has TMA stage the chunk's K and V rows (128-byte-swizzled tiles) into shared memory,
//   2. computes the logits of the G group heads on the tensor cores (mma.sync bf16, heads on the M
//      side with rows 8..15 duplicating rows 0..7), keeps them in shared memory in fp32,
//   3. forms p = 2^(s - chunk max), splits it into bf16 hi + lo parts that ride in rows 0..7 and
//      8..15 of the A operand, and accumulates the partial output  sum_j p_j v_j  (PV on tensor
//      cores, fp32 accumulate, hi and lo added afterwards: the product is exact to ~2^-17),
//   4. writes (max, sum, partial output) to global scratch and bumps the unit's arrival counter;
//      the CTA that arrives last merges the unit's partials into the final softmax statistics, the
//      attention output o and the reference vector X, and raises the unit's ready flag,
//   5. kLag chunks later - the chunk's V tile and logits are still resident in shared memory - waits
//      for that flag and writes c_j = w_j / (1 - w_j) * ||X - v_j|| for the chunk's tokens.
// So the second pass over V never leaves the SM. For the base modes that carry a score (ACCUM,
// EXTERNAL; G <= 7) row 7 of the A operand carries base_j, which yields sum_j base_j v_j for free.
//
// A CTA never waits before finishing step 4 of a chunk, and a unit's chunks all sit within one round
// of gridDim.x consecutive chunks (host-checked), so every wait of step 5 ends; each wait is
// nevertheless bounded by a clock limit, after which the kernel records CAOTE_ERR_TIMEOUT, stops
// waiting, drains its own copies and returns.
#pragma once

#include <cuda.h>

#include "common.cuh"

namespace caote {
namespace decode {

constexpr int kT = 128;             // tokens per chunk
constexpr int kLag = 2;             // chunks between a chunk's attention pass and its score pass
constexpr int kVBufs = kLag + 2;    // loading, attention pass, and kLag waiting for their unit
constexpr int kKBufs = 2;
constexpr int kSBufs = kLag + 1;
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kD = 128;
constexpr int kHalfBytes = kT * 128;  // one 64-channel box: kT rows of 128 bytes
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kRing = 256;            // chunk descriptors kept in shared memory
constexpr int kRefresh = 128;
constexpr long long kWaitCycles = 4000000000LL;  // ~2 s: far beyond any legitimate wait

struct PartialRec {   // per chunk
  float m[8];         // chunk max of the log2-domain logits per head
  float l[8];         // sum of 2^(s - m)
  float hb;           // sum of the carried base scores of the chunk
  float pad[7];
  float o[8][kD];     // sum_j p_j v_j per head (row 7: sum_j base_j v_j)
};
struct FinalRec {     // per unit
  float m[8];
  float inv_l[8];
  float H;            // normaliser of the base score: counted rows + sum of carried base scores
  float pad[7];
  float X[kD];
};
struct Desc {         // one chunk of this CTA's sequence
  int unit, lc, nchunks, pidx, n_valid, pad0, pad1, pad2;
};

struct Plan {
  int* chunk_prefix;  // [units + 1] exclusive prefix of chunks per unit
  int* counter;       // [units] chunks of the unit whose partials are written
  int* ready;         // [units] 1 once FinalRec is written
  PartialRec* part;   // [total chunks]
  FinalRec* fin;      // [units]
};

inline size_t carve(const Dims& dm, char* base, Plan* out) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    char* p = base + off;
    off = align_up(off + bytes, 256);
    return p;
  };
  Plan pl;
  const size_t max_chunks = (size_t)dm.units * ((dm.cap + kT - 1) / kT);
  pl.chunk_prefix = (int*)take(sizeof(int) * ((size_t)dm.units + 1));
  pl.counter = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.ready = (int*)take(sizeof(int) * (size_t)dm.units);
  pl.part = (PartialRec*)take(sizeof(PartialRec) * max_chunks);
  pl.fin = (FinalRec*)take(sizeof(FinalRec) * (size_t)dm.units);
  if (out) *out = pl;
  return off;
}

inline size_t smem_bytes() {
  return 1024 /* alignment slack */ + (size_t)(kKBufs + kVBufs) * kTileBytes + sizeof(float) * kSBufs * 8 * kT +
         16 * 32 * (kT / 16) /* P fragments */ + sizeof(float) * kSBufs * kT /* base */ + sizeof(Desc) * kRing +
         sizeof(FinalRec) + sizeof(float) * (kWarps * 8 * 2 + kT) + 256;
}

// ---- plan: chunks per unit, their prefix sum, and cleared counters / flags (one CTA) ------------
__global__ void __launch_bounds__(1024)
plan_kernel(int units, int Hkv, int cap, const int* __restrict__ len, Plan pl, int* status) {
  __shared__ int warp_tot[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) { carry = 0; pl.chunk_prefix[0] = 0; }
  __syncthreads();
  for (int u0 = 0; u0 < units; u0 += 1024) {
    const int u = u0 + tid;
    int nc = 0;
    if (u < units) {
      const int n = len[u / Hkv];
      if (n < 0 || n > cap) set_status(status, CAOTE_ERR_BAD_LENGTH);
      else nc = (n + kT - 1) / kT;
      pl.counter[u] = 0;
      pl.ready[u] = 0;
    }
    int incl = nc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int t = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    int before = carry;
    for (int w = 0; w < warp; ++w) before += warp_tot[w];
    if (u < units) pl.chunk_prefix[u + 1] = before + incl;
    __syncthreads();
    if (tid == 1023) carry = before + incl;
    __syncthreads();
  }
}

// ---- PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; returns false when the clock limit ran out.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > kWaitCycles) return false;
  return true;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_release(int* p, int v) {
  asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// bf16 hi/lo split of a non-negative float: x ~= hi + lo with ~16 significant bits.
__device__ __forceinline__ void split_pair(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(x0), h1 = __float2bfloat16_rn(x1);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(x0 - __bfloat162float(h0));
  const __nv_bfloat16 l1 = __float2bfloat16_rn(x1 - __bfloat162float(h1));
  hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}

// Byte offset of 16-byte chunk `chunk16` (0..15 along the 128 channels) of row `row` inside a staged
// tile: two 64-channel boxes, each kT rows x 128 bytes with the 128-byte swizzle (chunk ^ (row & 7)).
__device__ __forceinline__ uint32_t tile_off(int row, int chunk16) {
  return (uint32_t)((chunk16 >> 3) * kHalfBytes + row * 128 + (((chunk16 & 7) ^ (row & 7)) << 4));
}

__global__ void __launch_bounds__(kThreads, 1)
decode_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, Dims dm,
              const __nv_bfloat16* __restrict__ q, const int* __restrict__ len, float* __restrict__ base,
              float* __restrict__ o, float* __restrict__ scores, Plan pl, int* status) {
  extern __shared__ char smem_raw[];
  char* sm = reinterpret_cast<char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  char* Kbuf = sm;
  char* Vbuf = Kbuf + kKBufs * kTileBytes;
  float* Sbuf = reinterpret_cast<float*>(Vbuf + kVBufs * kTileBytes);   // [kSBufs][8][kT]
  uint4* Pbuf = reinterpret_cast<uint4*>(Sbuf + kSBufs * 8 * kT);       // [kT/16][32]
  float* Bbuf = reinterpret_cast<float*>(Pbuf + (kT / 16) * 32);        // [kSBufs][kT]
  Desc* ring = reinterpret_cast<Desc*>(Bbuf + kSBufs * kT);             // [kRing]
  FinalRec* frec = reinterpret_cast<FinalRec*>(ring + kRing);
  float* wmax = reinterpret_cast<float*>(frec + 1);                     // [kWarps][8]
  float* wl = wmax + kWarps * 8;                                        // [kWarps][8]
  float* nrm_s = wl + kWarps * 8;                                       // [kT]
  uint64_t* kbar = reinterpret_cast<uint64_t*>(nrm_s + kT);             // [kKBufs]
  uint64_t* vbar = kbar + kKBufs;                                       // [kVBufs]
  int* flags = reinterpret_cast<int*>(vbar + kVBufs);                   // [0] last arriver, [1] abort

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = dm.G, mode = dm.base_mode;
  const bool use_base = (mode == CAOTE_BASE_ACCUM || mode == CAOTE_BASE_EXTERNAL);
  const bool softmax_counted = (mode != CAOTE_BASE_EXTERNAL);
  const float scale2 = dm.scale * 1.4426950408889634f;  // logits are kept in the log2 domain

  const int total_chunks = pl.chunk_prefix[dm.units];
  const int my_iters = (total_chunks > (int)blockIdx.x)
                           ? (total_chunks - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
  if (my_iters == 0) return;

  if (tid == 0) {
    for (int i = 0; i < kKBufs; ++i) mbar_init(&kbar[i], 1);
    for (int i = 0; i < kVBufs; ++i) mbar_init(&vbar[i], 1);
    flags[0] = 0;
    flags[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }

  // chunk descriptors of iterations [first, first + count)
  auto fill_ring = [&](int first, int count) {
    for (int i = tid; i < count; i += kThreads) {
      const int it = first + i;
      Desc d;
      d.unit = -1;
      if (it < my_iters) {
        const int cid = (int)blockIdx.x + it * (int)gridDim.x;
        int lo = 0, hi = dm.units;  // largest u with prefix[u] <= cid
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (pl.chunk_prefix[mid] <= cid) lo = mid; else hi = mid;
        }
        const int p0 = pl.chunk_prefix[lo];
        d.unit = lo;
        d.lc = cid - p0;
        d.nchunks = pl.chunk_prefix[lo + 1] - p0;
        d.pidx = cid;
        d.n_valid = min(kT, len[lo / dm.Hkv] - d.lc * kT);
      }
      ring[it & (kRing - 1)] = d;
    }
  };
  fill_ring(0, kRefresh + 1);
  __syncthreads();

  auto issue_loads = [&](int it) {  // tid 0 only
    const Desc d = ring[it & (kRing - 1)];
    const int row = d.unit * dm.cap + d.lc * kT;
    char* kb = Kbuf + (it % kKBufs) * kTileBytes;
    char* vb = Vbuf + (it % kVBufs) * kTileBytes;
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    mbar_expect_tx(&kbar[it % kKBufs], kTileBytes);
    tma_load_2d(kb, &tmK, 0, row, &kbar[it % kKBufs]);
    tma_load_2d(kb + kHalfBytes, &tmK, 64, row, &kbar[it % kKBufs]);
    mbar_expect_tx(&vbar[it % kVBufs], kTileBytes);
    tma_load_2d(vb, &tmV, 0, row, &vbar[it % kVBufs]);
    tma_load_2d(vb + kHalfBytes, &tmV, 64, row, &vbar[it % kVBufs]);
  };
  if (tid == 0) issue_loads(0);
  int loads_issued = 1;  // iterations whose loads were issued (uniform across the CTA)
  bool aborted = false;

  for (int it = 0; it < my_iters + kLag; ++it) {
    __syncthreads();  // every buffer of iteration it - 1 is free to be reused
    if (flags[1]) { aborted = true; break; }
    if (it > 0 && (it % kRefresh) == 0) {
      fill_ring(it + 1, kRefresh);
      __syncthreads();
    }
    if (it + 1 < my_iters) {
      if (tid == 0) issue_loads(it + 1);
      loads_issued = it + 2;
    }

    if (it < my_iters) {
      // ===================== attention pass of chunk `it` =====================
      const Desc d = ring[it & (kRing - 1)];
      const int b = d.unit / dm.Hkv, h = d.unit % dm.Hkv;
      float* S = Sbuf + (it % kSBufs) * 8 * kT;
      float* Bb = Bbuf + (it % kSBufs) * kT;
      const uint32_t kaddr = smem_u32(Kbuf + (it % kKBufs) * kTileBytes);
      const uint32_t vaddr = smem_u32(Vbuf + (it % kVBufs) * kTileBytes);

      // Q fragments: row = lane / 4 (rows 8..15 duplicate rows 0..7), zero for heads >= G
      uint32_t qa[8][2];
      {
        const int g = lane >> 2;
        const __nv_bfloat16* qrow = q + ((size_t)b * dm.Hq + h * G + (g < G ? g : 0)) * kD + 2 * (lane & 3);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          qa[ks][0] = (g < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks) : 0u;
          qa[ks][1] = (g < G) ? *reinterpret_cast<const uint32_t*>(qrow + 16 * ks + 8) : 0u;
        }
      }
      if (tid < kT) Bb[tid] = (use_base && tid < d.n_valid) ? base[(size_t)d.unit * dm.cap + d.lc * kT + tid] : 0.f;

      if (!mbar_wait(&kbar[it % kKBufs], (it / kKBufs) & 1)) { flags[1] = 1; set_status(status, CAOTE_ERR_TIMEOUT); }

      // S = Q K^T for this warp's 16 tokens: two n-tiles of 8 tokens
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
      {
        const int mi = lane >> 3, r = lane & 7;
        const int tok = 16 * warp + 8 * (mi >> 1) + r;
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(kaddr + tile_off(tok, 2 * ks + (mi & 1)), b0, b1, b2, b3);
          mma_bf16(s0, qa[ks][0], qa[ks][0], qa[ks][1], qa[ks][1], b0, b1);
          mma_bf16(s1, qa[ks][0], qa[ks][0], qa[ks][1], qa[ks][1], b2, b3);
        }
      }
      // this thread: head = lane / 4, tokens t0, t0 + 1 (n-tile 0) and t0 + 8, t0 + 9 (n-tile 1)
      const int head = lane >> 2;
      const int t0 = 16 * warp + 2 * (lane & 3);
      float sv[4];
      sv[0] = (t0 < d.n_valid) ? s0[0] * scale2 : -INFINITY;
      sv[1] = (t0 + 1 < d.n_valid) ? s0[1] * scale2 : -INFINITY;
      sv[2] = (t0 + 8 < d.n_valid) ? s1[0] * scale2 : -INFINITY;
      sv[3] = (t0 + 9 < d.n_valid) ? s1[1] * scale2 : -INFINITY;
      *reinterpret_cast<float2*>(S + head * kT + t0) = make_float2(sv[0], sv[1]);
      *reinterpret_cast<float2*>(S + head * kT + t0 + 8) = make_float2(sv[2], sv[3]);
      float mx = fmaxf(fmaxf(sv[0], sv[1]), fmaxf(sv[2], sv[3]));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      if ((lane & 3) == 0) wmax[warp * 8 + head] = mx;
      __syncthreads();

      // chunk max, p, hi/lo split into the A fragments of k-step `warp`
      float mch = wmax[head];
#pragma unroll
      for (int w = 1; w < kWarps; ++w) mch = fmaxf(mch, wmax[w * 8 + head]);
      float p[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) p[i] = (sv[i] == -INFINITY) ? 0.f : exp2f(sv[i] - mch);
      float lsum = (p[0] + p[1]) + (p[2] + p[3]);
      lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
      lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
      if ((lane & 3) == 0) wl[warp * 8 + head] = lsum;
      if (head >= G) { p[0] = p[1] = p[2] = p[3] = 0.f; }
      if (use_base && head == 7) { p[0] = Bb[t0]; p[1] = Bb[t0 + 1]; p[2] = Bb[t0 + 8]; p[3] = Bb[t0 + 9]; }
      uint4 frag;  // a0 = hi(n-tile 0), a1 = lo(n-tile 0), a2 = hi(n-tile 1), a3 = lo(n-tile 1)
      split_pair(p[0], p[1], frag.x, frag.y);
      split_pair(p[2], p[3], frag.z, frag.w);
      Pbuf[warp * 32 + lane] = frag;

      if (!mbar_wait(&vbar[it % kVBufs], (it / kVBufs) & 1)) { flags[1] = 1; set_status(status, CAOTE_ERR_TIMEOUT); }
      if (d.n_valid < kT) {
        // rows behind the unit's length hold whatever the cache has there: clear them so that a
        // zero weight times a stray NaN cannot reach the accumulators
        char* vb = Vbuf + (it % kVBufs) * kTileBytes;
        const int rows = kT - d.n_valid;
        for (int i = tid; i < rows * 16; i += kThreads) {
          const int row = d.n_valid + (i >> 4), c = i & 15;
          *reinterpret_cast<uint4*>(vb + tile_off(row, c)) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      __syncthreads();

      // O^T slice: this warp owns channels [16 warp, 16 warp + 16), all kT tokens
      float o0[4] = {0.f, 0.f, 0.f, 0.f}, o1[4] = {0.f, 0.f, 0.f, 0.f};
      {
        const int mi = lane >> 3, r = lane & 7;
#pragma unroll
        for (int kk = 0; kk < kT / 16; ++kk) {
          const uint4 a = Pbuf[kk * 32 + lane];
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4_trans(vaddr + tile_off(16 * kk + 8 * (mi & 1) + r, 2 * warp + (mi >> 1)), b0, b1, b2, b3);
          mma_bf16(o0, a.x, a.y, a.z, a.w, b0, b1);
          mma_bf16(o1, a.x, a.y, a.z, a.w, b2, b3);
        }
      }
      PartialRec* pr = pl.part + d.pidx;
      {
        const int c0 = 16 * warp + 2 * (lane & 3);
        *reinterpret_cast<float2*>(&pr->o[head][c0]) = make_float2(o0[0] + o0[2], o0[1] + o0[3]);
        *reinterpret_cast<float2*>(&pr->o[head][c0 + 8]) = make_float2(o1[0] + o1[2], o1[1] + o1[3]);
      }
      if (warp == 0) {
        if (lane < 8) {
          float mm = wmax[lane], ll = wl[lane];
          for (int w = 1; w < kWarps; ++w) { mm = fmaxf(mm, wmax[w * 8 + lane]); ll += wl[w * 8 + lane]; }
          pr->m[lane] = mm;
          pr->l[lane] = ll;
        }
        float hb = (Bb[lane] + Bb[lane + 32]) + (Bb[lane + 64] + Bb[lane + 96]);
        hb = warp_sum(hb);
        if (lane == 0) pr->hb = hb;
      }
      __syncthreads();
      if (tid == 0) {
        __threadfence();
        const int old = atomicAdd(&pl.counter[d.unit], 1);
        flags[0] = (old == d.nchunks - 1);
      }
      __syncthreads();
      if (flags[0]) {
        // ---------- last arriver: merge the unit's partials ----------
        __threadfence();
        const PartialRec* p0 = pl.part + (d.pidx - d.lc);
        const int hd = tid >> 5, c4 = (tid & 31) * 4;
        const bool base_row = use_base && hd == 7;
        float mfin = -INFINITY;
        for (int c = 0; c < d.nchunks; ++c) mfin = fmaxf(mfin, __ldcg(&p0[c].m[hd]));
        float lfin = 0.f, hbsum = 0.f;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = 0; c < d.nchunks; ++c) {
          const float f = base_row ? 1.f : exp2f(__ldcg(&p0[c].m[hd]) - mfin);
          lfin = fmaf(__ldcg(&p0[c].l[hd]), f, lfin);
          const float4 v = __ldcg(reinterpret_cast<const float4*>(&p0[c].o[hd][c4]));
          acc.x = fmaf(v.x, f, acc.x);
          acc.y = fmaf(v.y, f, acc.y);
          acc.z = fmaf(v.z, f, acc.z);
          acc.w = fmaf(v.w, f, acc.w);
          hbsum += __ldcg(&p0[c].hb);
        }
        const float inv_l = (hd < G) ? 1.f / lfin : 0.f;
        float* xs = reinterpret_cast<float*>(Pbuf);  // [8][kD], free until the next iteration
        float4 contrib = make_float4(0.f, 0.f, 0.f, 0.f);
        if (hd < G) {
          const float4 on = make_float4(acc.x * inv_l, acc.y * inv_l, acc.z * inv_l, acc.w * inv_l);
          *reinterpret_cast<float4*>(o + ((size_t)b * dm.Hq + h * G + hd) * kD + c4) = on;
          if (softmax_counted) contrib = on;
        } else if (base_row) {
          contrib = acc;
        }
        *reinterpret_cast<float4*>(xs + hd * kD + c4) = contrib;
        FinalRec* fr = pl.fin + d.unit;
        const float Htot = (softmax_counted ? (float)G : 0.f) + (use_base ? hbsum : 0.f);
        if ((tid & 31) == 0) { fr->m[hd] = mfin; fr->inv_l[hd] = inv_l; }
        if (tid == 0) fr->H = Htot;
        __syncthreads();
        if (tid < kD) {
          float x = 0.f;
#pragma unroll
          for (int g = 0; g < 8; ++g) x += xs[g * kD + tid];
          fr->X[tid] = (Htot > 0.f) ? x / Htot : 0.f;
        }
        __syncthreads();
        if (tid == 0) {
          __threadfence();
          st_release(&pl.ready[d.unit], 1);
        }
      }
    }

    const int jt = it - kLag;
    if (jt >= 0 && jt < my_iters) {
      // ===================== score pass of chunk `jt` =====================
      const Desc d = ring[jt & (kRing - 1)];
      if (tid == 0) {
        const long long t0c = clock64();
        while (ld_acquire(&pl.ready[d.unit]) == 0) {
          if (clock64() - t0c > kWaitCycles) { flags[1] = 1; set_status(status, CAOTE_ERR_TIMEOUT); break; }
          __nanosleep(100);
        }
      }
      __syncthreads();
      if (flags[1]) { aborted = true; break; }
      if (tid < (int)(sizeof(FinalRec) / sizeof(float)))
        reinterpret_cast<float*>(frec)[tid] = __ldcg(reinterpret_cast<const float*>(pl.fin + d.unit) + tid);
      __syncthreads();
      const float* S = Sbuf + (jt % kSBufs) * 8 * kT;
      const float* Bb = Bbuf + (jt % kSBufs) * kT;
      const char* vb = Vbuf + (jt % kVBufs) * kTileBytes;
      const int row = tid & (kT - 1), half = tid >> 7;
      float acc = 0.f;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        const uint4 raw = *reinterpret_cast<const uint4*>(vb + tile_off(row, half * 8 + c));
        const uint32_t wv[4] = {raw.x, raw.y, raw.z, raw.w};
        const float* x = frec->X + half * 64 + c * 8;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&wv[e]));
          const float d0 = x[2 * e] - f.x, d1 = x[2 * e + 1] - f.y;
          acc = fmaf(d0, d0, acc);
          acc = fmaf(d1, d1, acc);
        }
      }
      if (half == 1) nrm_s[row] = acc;
      __syncthreads();
      if (half == 0 && row < d.n_valid) {
        acc += nrm_s[row];
        float hj = 0.f;
        if (softmax_counted) {
#pragma unroll
          for (int g = 0; g < 8; ++g)
            if (g < G) hj += exp2f(S[g * kT + row] - frec->m[g]) * frec->inv_l[g];
        }
        const size_t slot = (size_t)d.unit * dm.cap + d.lc * kT + row;
        if (mode == CAOTE_BASE_ACCUM) {
          hj += Bb[row];
          base[slot] = hj;
        } else if (mode == CAOTE_BASE_EXTERNAL) {
          hj = Bb[row];
        }
        const float Htot = frec->H;
        float ratio = 0.f;
        if (Htot > 0.f) {
          const float rest = Htot - hj;
          ratio = (rest > 0.f) ? hj / rest : INFINITY;
        }
        scores[slot] = (ratio == 0.f) ? 0.f : ((ratio == INFINITY) ? INFINITY : ratio * sqrtf(acc));
      }
    }
  }

  if (aborted) {
    // let this CTA's outstanding copies land before its shared memory goes away (bounded)
    __syncthreads();
    for (int it = 0; it < loads_issued; ++it) {
      if (it + kKBufs >= loads_issued) mbar_wait(&kbar[it % kKBufs], (it / kKBufs) & 1);
      if (it + kVBufs >= loads_issued) mbar_wait(&vbar[it % kVBufs], (it / kVBufs) & 1);
    }
  }
}

}  // namespace decode
}  // namespace caote
