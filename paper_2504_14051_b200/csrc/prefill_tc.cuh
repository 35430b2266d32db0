// Chunked-prefill scoring path on the 5th-generation tensor cores (tcgen05 + TMEM) for bf16,
// head_dim 128, base mode CHUNK_SUM: a block of m new queries per sequence, M = G * m query rows per
// (sequence, KV head) unit against its n cached keys.
//
//   attn_kernel   rows x keys. One CTA owns 128 query rows of a unit and walks the unit's keys in
//                 tiles of 128: S = Q K^T (tcgen05.mma, fp32 accumulator in TMEM), per-row online
//                 softmax straight out of TMEM (two threads per row, 64 keys each), P back into TMEM
//                 as two bf16 parts (hi + lo, 16 significant bits together), O += P V with P as the
//                 TMEM-side A operand and V as the MN-major B operand. Writes o and the per-row
//                 softmax statistics (reference, 1 / sum). One lane each of three extra warps issues
//                 the products, the K copies and the V copies, so the tensor pipe always has the
//                 next S queued while the rows are busy with the current one.
//   attn_combine_xsum_kernel   merges the key splits of small grids (attn_combine_kernel does only that, for
//                 FastCAOTE) and forms X = mean of the unit's M output rows (the weights of CHUNK_SUM are the
//                 column sums of the attention matrix divided by M, so sum_j w_j v_j is the mean output row).
//   score_kernel  keys x rows. One CTA owns 256 keys of a unit (two key tiles) and walks the unit's
//                 rows in blocks of 128: S^T = K Q^T lands in TMEM with one key per lane, so each
//                 thread sums exp2(s - ref_r) / sum_r over the rows of its own key without any
//                 exchange: h_j = sum_r alpha_{r,j}. Then c_j = w_j / (1 - w_j) * ||X - v_j||,
//                 w_j = h_j / M.
//
// Operands are staged by TMA as 64-channel boxes with the 128-byte swizzle, which is the canonical
// K-major UMMA layout (8-row groups 1024 bytes apart); V in the second product is read through an
// MN-major descriptor of the same bytes. Every mbarrier wait is bounded by a clock limit; a wait
// that runs out records CAOTE_ERR_TIMEOUT and the thread carries on with whatever is in its buffers
// (all indices stay in bounds), so that no thread is left behind at a barrier.
#pragma once

#include <cuda.h>

#include "common.cuh"
#include "ptx.cuh"

namespace caote {
namespace prefill {

constexpr int kD = 128;
constexpr int kTile = 128;                  // rows / keys per tile
constexpr int kHalfBytes = kTile * 128;     // one 64-channel box
constexpr int kTileBytes = 2 * kHalfBytes;  // 32 KB
constexpr int kThreads = 128;
constexpr long long kWaitCycles = 2000000000LL;

struct Scratch {
  float* stats;  // [units][Mpad]: log2-domain softmax reference + log2(sum of 2^(s - ref)): alpha = 2^(s - stats)
  float* X;      // [units][kD]
  int Mpad;      // M rounded up to a multiple of kTile
  int nsplit;    // key splits of the attention pass (1: none)
  float* po;     // [units][nsplit][Mpad][kD] per-split outputs, normalised by their own sums (nsplit > 1)
  float* pstat;  // [units][nsplit][Mpad] per-split statistics
};

// Few units and few query rows leave most SMs idle: the keys of a unit are then cut into up to 8 splits
// that run as CTAs of their own; attn_combine_kernel merges them. A function of the shape only.
inline int attn_splits(const Dims& dm) {
  const long long ctas = (long long)((dm.R + kTile - 1) / kTile) * dm.units;
  long long ns = g_sm_count / (ctas > 0 ? ctas : 1);
  const long long max_by_len = ((dm.cap + kTile - 1) / kTile) / 4;  // at least four tiles per split
  if (ns > max_by_len) ns = max_by_len;
  if (ns > 8) ns = 8;
  return ns < 1 ? 1 : (int)ns;
}
// Split plan for a unit of n keys, the last m of them new (device and host agree on it): `ts` tiles per
// split, `count` splits in use. The new block must lie inside the last split, so that every row sees at
// least one key in every split it takes part in.
__host__ __device__ inline void split_plan(int n, int m, int nsplit, int& ts, int& count) {
  const int ntiles = (n + kTile - 1) / kTile;
  for (int k = nsplit; k >= 1; --k) {
    ts = (ntiles + k - 1) / k;
    count = (ntiles + ts - 1) / ts;
    if ((count - 1) * ts * kTile <= n - m) return;
  }
  ts = ntiles;
  count = 1;
}

inline size_t carve(const Dims& dm, char* base, Scratch* out) {
  Scratch s;
  s.Mpad = (dm.R + kTile - 1) / kTile * kTile;
  size_t off = 0;
  s.stats = reinterpret_cast<float*>(base + off);
  off = align_up(off + sizeof(float) * (size_t)dm.units * s.Mpad, 256);
  s.X = reinterpret_cast<float*>(base + off);
  off = align_up(off + sizeof(float) * (size_t)dm.units * kD, 256);
  s.nsplit = attn_splits(dm);
  s.po = s.pstat = nullptr;
  if (s.nsplit > 1) {
    s.po = reinterpret_cast<float*>(base + off);
    off = align_up(off + sizeof(float) * (size_t)dm.units * s.nsplit * s.Mpad * kD, 256);
    s.pstat = reinterpret_cast<float*>(base + off);
    off = align_up(off + sizeof(float) * (size_t)dm.units * s.nsplit * s.Mpad, 256);
  }
  if (out) *out = s;
  return off;
}

// ---- PTX wrappers (ptx.cuh), the waits built on them, and the tcgen05 wrappers ----------------------------
using ptx::smem_u32;
using ptx::mbar_init;
using ptx::mbar_expect_tx;
using ptx::mbar_arrive;
using ptx::mbar_try_wait;
using ptx::tma_load_2d;
using ptx::bulk_load;
using ptx::fence_async_smem;
using ptx::fast_exp2;
using ptx::tile_off;
// Bounded wait. On expiry the error is recorded and the caller carries on (see the file comment).
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      return;
    }
  }
}
// The same for the single-lane helper warps: they back off between polls so that their spinning does
// not take issue slots from the warps that do the arithmetic on the same scheduler.
__device__ __forceinline__ void mbar_wait_idle(uint64_t* bar, uint32_t parity, int* status) {
  if (mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    __nanosleep(20);
    if (clock64() - t0 > kWaitCycles) {
      set_status(status, CAOTE_ERR_TIMEOUT);
      return;
    }
  }
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// TMEM: `cols` columns (a power of two >= 32) for this CTA; one warp allocates, the same warp frees.
__device__ __forceinline__ void tmem_alloc(uint32_t* slot_in_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// Shared-memory matrix descriptor (bf16 tiles staged as 128-byte rows with the 128-byte swizzle).
//   bits [0,14)  start address >> 4        bits [16,30) leading byte offset >> 4
//   bits [32,46) stride byte offset >> 4   bits [46,48) descriptor version (1 on sm_100)
//   bits [61,64) layout type (2 = 128-byte swizzle)
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of tcgen05.mma.kind::f16: bf16 x bf16 -> fp32, M = 128, N = 128.
//   bits [4,6) D format (1 = f32), [7,10) A format (1 = bf16), [10,13) B format (1 = bf16),
//   bit 15 A major, bit 16 B major (0 = K-major, 1 = MN-major), [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t instr_desc(bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]; issued by one thread.
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
// The mbarrier gets one arrival once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// The same load without the wait, and the wait as a statement that the 32 registers pass through: whatever reads
// them afterwards depends on the wait, so the compiler cannot move such a read in front of it. Between the two
// the thread may do anything that does not touch r.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld32_wait(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
        "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
        "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
        "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
      :: "memory");
}
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld16_wait(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
      : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
        "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
      :: "memory");
}
// Sixteen floats from shared memory, issued where the statement stands (the compiler may not sink it towards the
// first use: the point is to have the loads in flight while other work is done).
__device__ __forceinline__ void lds16_issue(const float* p, float4 (&s)[4]) {
  const uint32_t a = smem_u32(p);
#pragma unroll
  for (int k = 0; k < 4; ++k)
    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(s[k].x), "=f"(s[k].y), "=f"(s[k].z), "=f"(s[k].w) : "r"(a + 16 * k));
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])),
        "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])),
        "r"(__float_as_uint(v[19])), "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])),
        "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])),
        "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])),
        "r"(__float_as_uint(v[31])) : "memory");
}
__device__ __forceinline__ void tmem_st32u(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]),
        "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]),
        "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31]) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]: the A operand (K-major, two bf16 per 32-bit column) comes from TMEM.
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.u32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"((uint32_t)accumulate) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ uint32_t pack_bf16(float x0, float x1) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(x1), "f"(x0));
  return r;
}
// Descriptors of k-step ks (16 of the 128 contraction elements) of a staged tile.
//   K-major: contraction along the 128-byte rows: 32 bytes per step inside a box, second box after 4.
//   MN-major: contraction along the rows of the tile (16 rows = 2 groups of 8 = 2048 bytes per
//   step); the two 64-element boxes along MN are kHalfBytes apart (leading byte offset).
__device__ __forceinline__ uint64_t desc_k_major(uint32_t tile_addr, int ks) {
  return smem_desc(tile_addr + (ks >> 2) * kHalfBytes + (ks & 3) * 32, 16, 1024);
}
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t tile_addr, int ks) {
  return smem_desc(tile_addr + ks * 2048, kHalfBytes, 1024);
}


// ---- attention pass ---------------------------------------------------------------------------------
// Keys are walked in tiles of 128: three K stages, two V stages and the Q block in shared memory, two S buffers,
// and O in TMEM, P (bf16 hi and lo parts) written over the S it came from; the tensor pipe then always has the next
// S = Q K^T queued while the threads are busy with the softmax of the current tile:
//   tensor pipe:  QK(t+1)  PV(t)  QK(t+2)  PV(t+1) ...
//   threads:      softmax(t) ............ softmax(t+1) ...
constexpr int kKeys = 128;                   // keys per tile of the attention pass
constexpr int kKvHalf = kKeys * 128;         // one 64-channel box of 128 keys: 16 KB
constexpr int kKvTile = 2 * kKvHalf;         // K or V tile: 32 KB
constexpr int kKStages = 3;                  // a K stage is free as soon as S is formed
constexpr int kVStages = 2;
constexpr int kRowThreads = 2 * kThreads;    // two threads per query row: each owns 64 of the tile's 128 keys
constexpr int kAttnThreads = kRowThreads + 96;  // + MMA, K-load and V-load warps

inline size_t attn_smem_bytes() {
  return 1024 + kTileBytes + (size_t)(kKStages + kVStages) * kKvTile + 2 * kRowThreads * sizeof(float) + 256;
}

// K-major / MN-major descriptors of k-step ks of a key tile (boxes of kKeys rows x 64 channels: kKvHalf apart).
__device__ __forceinline__ uint64_t desc_k_major64(uint32_t tile_addr, int ks) {
  return smem_desc(tile_addr + (ks >> 2) * kKvHalf + (ks & 3) * 32, 16, 1024);
}
__device__ __forceinline__ uint64_t desc_mn_major64(uint32_t tile_addr, int ks) {
  return smem_desc(tile_addr + ks * 2048, kKvHalf, 1024);
}
__host__ __device__ constexpr uint32_t instr_desc_n(bool b_mn_major, uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((b_mn_major ? 1u : 0u) << 16) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// o and row statistics of 128 query rows of one unit. grid = (row blocks, units), 352 threads:
// warps 0..7 are the row threads (two per row); one lane each of warps 8, 9, 10 issues the products,
// the K copies and the V copies.
// tmK64 / tmV64: tensor maps of K and V with boxes of 64 channels x kKeys rows.
__global__ void __launch_bounds__(kAttnThreads, 1)
attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK64,
            const __grid_constant__ CUtensorMap tmV64, Dims dm, const int* __restrict__ len, Scratch sc,
            float* __restrict__ o, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  extern __shared__ char smem_raw[];
  // (aligned by an offset into the array, not through an integer: the pointer keeps its address space, and what is
  // read and written through it compiles to shared-memory accesses, not generic ones)
  char* sm = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  char* Qs = sm;
  char* Ksm = Qs + kTileBytes;                 // [kKStages]
  char* Vsm = Ksm + kKStages * kKvTile;        // [kVStages]
  float* xch = reinterpret_cast<float*>(Vsm + kVStages * kKvTile);  // [2][kRowThreads] half-row maxima / sums
  uint64_t* bars = reinterpret_cast<uint64_t*>(xch + 2 * kRowThreads);
  uint64_t *q_bar = &bars[0], *k_bar = &bars[1], *v_bar = k_bar + kKStages, *s_bar = v_bar + kVStages, *o_bar = s_bar + 2,
           *p_bar = o_bar + 2, *k_free = p_bar + 2, *v_free = k_free + kKStages;
  constexpr int kBars = 1 + 2 * (kKStages + kVStages) + 6;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kBars);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int unit = blockIdx.y, row0 = blockIdx.x * kTile;
  const int b = unit / dm.Hkv;
  const int n = len[b], M = dm.R, m = dm.m;
  if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) status[kStatTagIndex] = kStatPerRow;
  if (n == 0) return;
  if (n < m || n > dm.cap) {
    if (tid == 0) set_status(status, CAOTE_ERR_BAD_LENGTH);
    return;
  }
  // this CTA's share of the unit's key tiles: [kt0, kt0 + ntiles)
  int ts, nsp;
  split_plan(n, m, sc.nsplit, ts, nsp);
  const int split = blockIdx.z;
  if (split >= nsp) return;
  const int kt0 = split * ts;
  const int ntiles = min(ts, (n + kKeys - 1) / kKeys - kt0);

  if (tid == 0) {
    for (int i = 0; i < kBars; ++i) mbar_init(&bars[i], 1);
    mbar_init(&p_bar[0], kRowThreads);
    mbar_init(&p_bar[1], kRowThreads);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  // columns: S0 [0,128), S1 [128,256), O [256,384). P of a tile takes the place of its S once the row threads have
  // read that: hi part in the buffer's columns [0,64), lo part in [64,128) (two bf16 per column), so P is double-
  // buffered like S and the softmax of a tile does not wait for the previous tile's O += P V
  const uint32_t tmem = *tmem_slot;

  if (warp == 9) {
    // =============================== K loads (one lane) ===============================
    if (tid == kRowThreads + 32) {
      mbar_expect_tx(q_bar, kTileBytes);
      tma_load_2d(Qs, &tmQ, 0, unit * M + row0, q_bar);
      tma_load_2d(Qs + kHalfBytes, &tmQ, 64, unit * M + row0, q_bar);
      for (int kt = 0; kt < ntiles; ++kt) {
        const int st = kt % kKStages, row = unit * dm.cap + (kt0 + kt) * kKeys;
        if (kt >= kKStages) mbar_wait_idle(&k_free[st], ((kt / kKStages) - 1) & 1, status);  // S of tile kt - 3 is formed
        mbar_expect_tx(&k_bar[st], kKvTile);
        tma_load_2d(Ksm + st * kKvTile, &tmK64, 0, row, &k_bar[st]);
        tma_load_2d(Ksm + st * kKvTile + kKvHalf, &tmK64, 64, row, &k_bar[st]);
      }
    }
  } else if (warp == 10) {
    // =============================== V loads (one lane) ===============================
    if (tid == kRowThreads + 64) {
      for (int kt = 0; kt < ntiles; ++kt) {
        const int st = kt % kVStages, row = unit * dm.cap + (kt0 + kt) * kKeys;
        if (kt >= kVStages) mbar_wait_idle(&v_free[st], ((kt / kVStages) - 1) & 1, status);  // O += P V of tile kt - 2 is done
        mbar_expect_tx(&v_bar[st], kKvTile);
        tma_load_2d(Vsm + st * kKvTile, &tmV64, 0, row, &v_bar[st]);
        tma_load_2d(Vsm + st * kKvTile + kKvHalf, &tmV64, 64, row, &v_bar[st]);
      }
    }
  } else if (warp == 8) {
    // =============================== products (one lane) ===============================
    if (tid == kRowThreads) {
      constexpr uint32_t kIdescS = instr_desc_n(false, kKeys), kIdescO = instr_desc_n(true, kD);
      const uint32_t q_addr = smem_u32(Qs);
      // Descriptors are built once; inside the loop a product costs one 64-bit add per operand (the
      // single issuing thread is bound by the latency of its own instruction stream, not by the pipe).
      uint64_t qdesc[8];
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) qdesc[ks] = desc_k_major(q_addr, ks);
      const uint64_t kdesc0 = smem_desc(smem_u32(Ksm), 16, 1024);
      const uint64_t vdesc0 = smem_desc(smem_u32(Vsm), kKvHalf, 1024);
      auto issue_qk = [&](int kt) {
        mbar_wait_idle(&k_bar[kt % kKStages], (kt / kKStages) & 1, status);
        tc_fence_after();
        const uint64_t kd = kdesc0 + (uint64_t)(((kt % kKStages) * kKvTile) >> 4);
        const uint32_t d_s = tmem + (kt & 1) * kKeys;  // S0 or S1
#pragma unroll
        for (int ks = 0; ks < 8; ++ks)
          umma(d_s, qdesc[ks], kd + (uint64_t)((((ks >> 2) * kKvHalf) + (ks & 3) * 32) >> 4), kIdescS, ks > 0);
        umma_commit(&s_bar[kt & 1]);
        umma_commit(&k_free[kt % kKStages]);
      };
      mbar_wait_idle(q_bar, 0, status);
      issue_qk(0);
      for (int kt = 0; kt < ntiles; ++kt) {
        // queue S of the next tile: its buffer was read by the softmax of tile kt - 1, which has
        // arrived on p_bar before PV(kt - 1) was issued
        if (kt + 1 < ntiles) issue_qk(kt + 1);
        // O += P V once the rows have written P of this tile
        mbar_wait_idle(&p_bar[kt & 1], (kt >> 1) & 1, status);
        mbar_wait_idle(&v_bar[kt % kVStages], (kt / kVStages) & 1, status);
        tc_fence_after();
        const uint64_t vd = vdesc0 + (uint64_t)(((kt % kVStages) * kKvTile) >> 4);
        const uint32_t p_tmem = tmem + (kt & 1) * kKeys;
        if (kt == 0) {
          umma_ts(tmem + 256, p_tmem, vd, kIdescO, false);
        } else {
          umma_ts(tmem + 256, p_tmem, vd, kIdescO, true);
        }
        umma_ts(tmem + 256, p_tmem + 64, vd, kIdescO, true);
#pragma unroll
        for (int ks = 1; ks < 8; ++ks) {  // 16 keys = 8 packed columns per step
          umma_ts(tmem + 256, p_tmem + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), kIdescO, true);
          umma_ts(tmem + 256, p_tmem + 64 + ks * 8, vd + (uint64_t)((ks * 2048) >> 4), kIdescO, true);
        }
        umma_commit(&o_bar[kt & 1]);
        umma_commit(&v_free[kt % kVStages]);
      }
    }
  } else {
    // =============================== two threads per query row ===============================
    // Thread t and thread t + 128 share row t of the block: each owns 64 of a tile's 128 keys (and 64
    // of the 128 output channels when O is rescaled or written out). They agree on the softmax
    // reference through a two-float exchange in shared memory and one barrier of the row threads.
    const int rowl = tid & (kThreads - 1), half = tid >> 7;
    const int R = row0 + rowl;
    const int nvis = (R < M) ? n - m + (R % m) + 1 : n;  // keys this row sees (causal inside the block)
    const float scale2 = dm.scale * 1.4426950408889634f;
    const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t t_o = t_lane + 256 + half * 64;
    float m_ref = -INFINITY, l = 0.f;

    for (int kt = 0; kt < ntiles; ++kt) {
      mbar_wait(&s_bar[kt & 1], (kt >> 1) & 1, status);
      tc_fence_after();
      const int j0 = (kt0 + kt) * kKeys + half * 64;  // first key of this thread's half
      const uint32_t t_s = t_lane + (kt & 1) * kKeys + half * 64;
      float sv[64];  // raw products; masked keys become -inf
      tmem_ld32(t_s, *reinterpret_cast<float(*)[32]>(&sv[0]));
      tmem_ld32(t_s + 32, *reinterpret_cast<float(*)[32]>(&sv[32]));
      if ((kt0 + kt) * kKeys + kKeys > n - m + 1) {  // only tiles that reach into the new block (or past the length) need the mask
#pragma unroll
        for (int i = 0; i < 64; ++i) sv[i] = (j0 + i < nvis) ? sv[i] : -INFINITY;
      }
      float mx;
      {
        float pm[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) pm[i] = sv[i] * scale2;
#pragma unroll
        for (int i = 8; i < 64; ++i) pm[i & 7] = fmaxf(pm[i & 7], sv[i] * scale2);
        mx = fmaxf(fmaxf(fmaxf(pm[0], pm[1]), fmaxf(pm[2], pm[3])), fmaxf(fmaxf(pm[4], pm[5]), fmaxf(pm[6], pm[7])));
      }
      // the other half of the row
      float* xm = xch + (kt & 1) * kRowThreads;
      xm[tid] = mx;
      asm volatile("bar.sync 1, %0;" ::"n"(kRowThreads) : "memory");
      mx = fmaxf(mx, xm[tid ^ kThreads]);
      // the reference moves only when a logit exceeds it by more than 8 (p <= 256 in between)
      const bool need = mx > m_ref + 8.f;
      if (__any_sync(0xffffffffu, need)) {
        const float corr = need ? fast_exp2(m_ref - mx) : 1.f;
        if (need) m_ref = mx;
        l *= corr;
        if (kt > 0) {
          mbar_wait(&o_bar[(kt - 1) & 1], ((kt - 1) >> 1) & 1, status);  // O += P V of the previous tile is done
          tc_fence_after();
#pragma unroll
          for (int cc = 0; cc < 2; ++cc) {
            float v[32];
            tmem_ld32(t_o + cc * 32, v);
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] *= corr;
            tmem_st32(t_o + cc * 32, v);
          }
          tmem_st_wait();
        }
      }
      {
        const float neg_ref = -m_ref;
        float ls[4] = {0.f, 0.f, 0.f, 0.f};
        uint32_t hi[32], lo[32];  // column c = keys 2c (low half) and 2c + 1
#pragma unroll
        for (int c = 0; c < 32; ++c) {
          // P = hi + lo, hi truncated and lo rounded to bf16 (16 significant bits together); plain bit
          // operations, so the conversion unit is left to the exponentials
          const float p0 = fast_exp2(fmaf(sv[2 * c], scale2, neg_ref));
          const float p1 = fast_exp2(fmaf(sv[2 * c + 1], scale2, neg_ref));
          const uint32_t b0 = __float_as_uint(p0), b1 = __float_as_uint(p1);
          hi[c] = __byte_perm(b0, b1, 0x7632);
          const float r0 = p0 - __uint_as_float(b0 & 0xffff0000u), r1 = p1 - __uint_as_float(b1 & 0xffff0000u);
          lo[c] = __byte_perm(__float_as_uint(r0) + 0x8000u, __float_as_uint(r1) + 0x8000u, 0x7632);  // rounded
          ls[c & 3] += p0 + p1;
        }
        // P goes where S was: both halves of the row have read their S columns (the barrier above), and the
        // product that read the buffer's previous P was issued before the product that formed this S
        const uint32_t t_p = t_lane + (kt & 1) * kKeys + half * 32;  // this half's 64 keys = 32 packed columns
        tmem_st32u(t_p, hi);
        tmem_st32u(t_p + 64, lo);
        tmem_st_wait();
        l += (ls[0] + ls[1]) + (ls[2] + ls[3]);
      }
      const int n_valid = min(kKeys, n - (kt0 + kt) * kKeys);
      if (n_valid < kKeys) {
        // V rows behind the unit's length: clear them so that 0 * (stray NaN) cannot reach O
        mbar_wait(&v_bar[kt % kVStages], (kt / kVStages) & 1, status);
        if (tid < kKeys && tid >= n_valid) {
          char* vt = Vsm + (kt % kVStages) * kKvTile;
#pragma unroll
          for (int c = 0; c < 16; ++c)
            *reinterpret_cast<uint4*>(vt + (c >> 3) * kKvHalf + tid * 128 + (((c & 7) ^ (tid & 7)) << 4)) = make_uint4(0u, 0u, 0u, 0u);
        }
      }
      fence_async_smem();
      tc_fence_before();
      mbar_arrive(&p_bar[kt & 1]);
    }
    mbar_wait(&o_bar[(ntiles - 1) & 1], ((ntiles - 1) >> 1) & 1, status);
    tc_fence_after();

    // ---- normalise and write out: the two halves of a row add up their sums first ----
    float* xl = xch + (ntiles & 1) * kRowThreads;  // the copy the last tile did not use
    xl[tid] = l;
    asm volatile("bar.sync 1, %0;" ::"n"(kRowThreads) : "memory");
    l += xl[tid ^ kThreads];
    const float inv_l = 1.f / l;
    // (with key splits: this split's output, normalised by its own sum, and its statistic go to scratch)
    float* orow = (nsp > 1 ? sc.po + (((size_t)unit * sc.nsplit + split) * sc.Mpad + R) * kD
                           : o + ((size_t)unit * M + R) * kD) + half * 64;
#pragma unroll
    for (int cc = 0; cc < 2; ++cc) {
      float v[32];
      tmem_ld32(t_o + cc * 32, v);  // collective: every lane takes part, rows beyond M just do not store
      if (R < M) {
#pragma unroll
        for (int i = 0; i < 32; i += 4)
          *reinterpret_cast<float4*>(orow + cc * 32 + i) = make_float4(v[i] * inv_l, v[i + 1] * inv_l, v[i + 2] * inv_l, v[i + 3] * inv_l);
      }
    }
    if (R < M && half == 0) {
      if (nsp > 1) sc.pstat[((size_t)unit * sc.nsplit + split) * sc.Mpad + R] = m_ref + __log2f(l);
      else sc.stats[(size_t)unit * sc.Mpad + R] = m_ref + __log2f(l);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

// Merge the key splits of a unit: o = sum_s o_s 2^(stat_s - stat), stat = log2 sum_s 2^stat_s.
// grid = (ceil(M / 4), units), 4 rows x 128 channels per CTA. Units that ran unsplit are left alone.
__global__ void __launch_bounds__(4 * kD)
attn_combine_kernel(Dims dm, const int* __restrict__ len, Scratch sc, float* __restrict__ o) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  const int unit = blockIdx.y, c = threadIdx.x % kD, R = blockIdx.x * 4 + threadIdx.x / kD;
  const int n = len[unit / dm.Hkv];
  if (n == 0 || n < dm.m || n > dm.cap || R >= dm.R) return;
  int ts, nsp;
  split_plan(n, dm.m, sc.nsplit, ts, nsp);
  if (nsp <= 1) return;
  float st[8], mx = -INFINITY;
  for (int s = 0; s < nsp; ++s) {
    st[s] = sc.pstat[((size_t)unit * sc.nsplit + s) * sc.Mpad + R];
    mx = fmaxf(mx, st[s]);
  }
  float tot = 0.f, acc = 0.f;
  for (int s = 0; s < nsp; ++s) {
    const float w = exp2f(st[s] - mx);
    tot += w;
    acc = fmaf(sc.po[(((size_t)unit * sc.nsplit + s) * sc.Mpad + R) * kD + c], w, acc);
  }
  o[((size_t)unit * dm.R + R) * kD + c] = acc / tot;
  if (c == 0) sc.stats[(size_t)unit * sc.Mpad + R] = mx + log2f(tot);
}

// The merge of the key splits and the column mean X (the weights of CHUNK_SUM are the column sums of the attention
// matrix divided by M, so sum_j w_j v_j is the mean output row) in one launch: a CTA takes 16 channels of a unit and
// all of its rows, merges the splits row by row exactly as attn_combine_kernel does, writes o and (the CTA of channels
// 0..15) the rows' statistics, and adds up its 16 columns in a fixed order for X. Units that ran unsplit are only
// summed. grid = (units, kD / 16), 512 threads: a warp takes 8 rows at a time, 4 lanes per row.
constexpr int kCxThreads = 512;
__global__ void __launch_bounds__(kCxThreads, 2)
attn_combine_xsum_kernel(Dims dm, const int* __restrict__ len, Scratch sc, float* __restrict__ o) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  __shared__ float4 wpart[kCxThreads / 32][4];
  const int unit = blockIdx.x, c0 = blockIdx.y * 16;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n = len[unit / dm.Hkv];
  if (n == 0 || n < dm.m || n > dm.cap) return;
  int ts, nsp;
  split_plan(n, dm.m, sc.nsplit, ts, nsp);
  const int ch = c0 + 4 * (lane & 3);
  float4 cs = make_float4(0.f, 0.f, 0.f, 0.f);
  // A warp's time here is round trips to L2, not arithmetic: every load of a pass is issued before the first use.
  constexpr int kStep = (kCxThreads / 32) * 8;
  if (nsp > 1) {
    // (splits beyond nsp count as weight zero, which leaves every sum as it is)
    for (int R = warp * 8 + (lane >> 2); R < dm.R; R += kStep) {
      float st[8];
      float4 p[8];
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        st[s] = -INFINITY;
        p[s] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (s < nsp) {
          st[s] = sc.pstat[((size_t)unit * sc.nsplit + s) * sc.Mpad + R];
          p[s] = *reinterpret_cast<const float4*>(sc.po + (((size_t)unit * sc.nsplit + s) * sc.Mpad + R) * kD + ch);
        }
      }
      float mx = -INFINITY;
#pragma unroll
      for (int s = 0; s < 8; ++s) mx = fmaxf(mx, st[s]);
      float tot = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int s = 0; s < 8; ++s) {
        const float w = (s < nsp) ? exp2f(st[s] - mx) : 0.f;
        tot += w;
        acc.x = fmaf(p[s].x, w, acc.x); acc.y = fmaf(p[s].y, w, acc.y);
        acc.z = fmaf(p[s].z, w, acc.z); acc.w = fmaf(p[s].w, w, acc.w);
      }
      const float4 res = make_float4(acc.x / tot, acc.y / tot, acc.z / tot, acc.w / tot);
      *reinterpret_cast<float4*>(o + ((size_t)unit * dm.R + R) * kD + ch) = res;
      if (ch == 0) sc.stats[(size_t)unit * sc.Mpad + R] = mx + log2f(tot);
      cs.x += res.x; cs.y += res.y; cs.z += res.z; cs.w += res.w;
    }
  } else {
    for (int R0 = warp * 8 + (lane >> 2); R0 < dm.R; R0 += 4 * kStep) {  // four rows in flight, summed in row order
      float4 r[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int R = R0 + u * kStep;
        r[u] = (R < dm.R) ? *reinterpret_cast<const float4*>(o + ((size_t)unit * dm.R + R) * kD + ch)
                          : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
        if (R0 + u * kStep < dm.R) { cs.x += r[u].x; cs.y += r[u].y; cs.z += r[u].z; cs.w += r[u].w; }
    }
  }
  // the warp's eight row lanes of every channel quad, then the warps in order
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    cs.x += __shfl_xor_sync(0xffffffffu, cs.x, off);
    cs.y += __shfl_xor_sync(0xffffffffu, cs.y, off);
    cs.z += __shfl_xor_sync(0xffffffffu, cs.z, off);
    cs.w += __shfl_xor_sync(0xffffffffu, cs.w, off);
  }
  if (lane < 4) wpart[warp][lane] = cs;
  __syncthreads();
  if (tid < 4) {
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int w = 0; w < kCxThreads / 32; ++w) {
      const float4 p = wpart[w][tid];
      t.x += p.x; t.y += p.y; t.z += p.z; t.w += p.w;
    }
    const float inv = 1.f / (float)dm.R;
    *reinterpret_cast<float4*>(sc.X + (size_t)unit * kD + c0 + 4 * tid) = make_float4(t.x * inv, t.y * inv, t.z * inv, t.w * inv);
  }
}

constexpr int kScoreKeys = 2 * kTile;            // keys per CTA: two key tiles share every Q block
constexpr int kKeyThreads = 2 * kScoreKeys;       // two threads per key: each owns 64 of a block's 128 rows
constexpr int kScoreThreads = kKeyThreads + 64;   // + a warp for the products + a warp for the copies
constexpr int kStatBytes = kTile * 4;             // the softmax statistic of the 128 rows of a block
constexpr int kQStages = 4;                       // Q blocks: a stage is free again once its products are done
constexpr int kSStages = 8;                       // their rows' statistics: free once the key threads have used them

inline size_t score_smem_bytes() {
  return 1024 + (2 + kQStages) * (size_t)kTileBytes + kSStages * (size_t)kStatBytes + (kD + kScoreKeys) * sizeof(float) + 256;
}

// 2^x for two arguments at once on the FMA pipe instead of the special-function unit: x = i + f with i the nearest
// integer (taken from the low bits of x + 1.5 * 2^23), 2^f on [-1/2, 1/2] by a polynomial of degree 4 that is exact at
// f = 0 (relative error below 3e-6), and i added to the exponent field. Arguments below -126 give about 2^-126.
// The score pass is bound by the special-function unit's 16 results per clock and SM (one exponential per
// (row, key) pair); it hands a quarter of them to this routine.
__device__ __forceinline__ float2 poly_exp2x2(float2 x) {
  constexpr float kMagic = 12582912.f;
  x.x = fmaxf(x.x, -126.f);
  x.y = fmaxf(x.y, -126.f);
  const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 r = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
  const float2 f = __ffma2_rn(r, make_float2(-1.f, -1.f), x);
  float2 p = __ffma2_rn(make_float2(0.009589649736881256f, 0.009589649736881256f), f,
                        make_float2(0.05590599775314331f, 0.05590599775314331f));
  p = __ffma2_rn(p, f, make_float2(0.24023915827274323f, 0.24023915827274323f));
  p = __ffma2_rn(p, f, make_float2(0.6931241154670715f, 0.6931241154670715f));
  p = __ffma2_rn(p, f, make_float2(1.f, 1.f));
  return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}

// Adds to a key's running sum the attention weights 2^(s * scale2 - statistic) of 16 rows (v: the logits of the
// key against these rows, st: the rows' statistics). plain: no row is masked. Of every eight exponentials six go to
// the special-function unit and two to the polynomial.
__device__ __forceinline__ void score_piece16(const uint32_t (&v)[16], const float4 (&st)[4], float scale2, bool plain,
                                              int R0, int M, int m, int need, float2 (&hacc)[2], float& hmasked) {
  if (plain) {
#pragma unroll
    for (int i = 0; i < 16; i += 8) {
      const float4 ra = st[i / 4], rb = st[i / 4 + 1];
      const float a0 = fast_exp2(fmaf(__uint_as_float(v[i]), scale2, -ra.x));
      const float a1 = fast_exp2(fmaf(__uint_as_float(v[i + 1]), scale2, -ra.y));
      const float a2 = fast_exp2(fmaf(__uint_as_float(v[i + 2]), scale2, -ra.z));
      const float a3 = fast_exp2(fmaf(__uint_as_float(v[i + 3]), scale2, -ra.w));
      const float a4 = fast_exp2(fmaf(__uint_as_float(v[i + 4]), scale2, -rb.x));
      const float a5 = fast_exp2(fmaf(__uint_as_float(v[i + 5]), scale2, -rb.y));
      const float2 a67 = poly_exp2x2(make_float2(fmaf(__uint_as_float(v[i + 6]), scale2, -rb.z),
                                                 fmaf(__uint_as_float(v[i + 7]), scale2, -rb.w)));
      hacc[0] = __fadd2_rn(hacc[0], make_float2(a0, a1));
      hacc[1] = __fadd2_rn(hacc[1], make_float2(a2, a3));
      hacc[0] = __fadd2_rn(hacc[0], make_float2(a4, a5));
      hacc[1] = __fadd2_rn(hacc[1], a67);
    }
  } else {
    // row R sees key j iff j <= n - m + (R % m), i.e. iff (R % m) >= need; R % m is carried along instead of
    // being divided out for every pair
    const float stf[16] = {st[0].x, st[0].y, st[0].z, st[0].w, st[1].x, st[1].y, st[1].z, st[1].w,
                           st[2].x, st[2].y, st[2].z, st[2].w, st[3].x, st[3].y, st[3].z, st[3].w};
    int rm = R0 % m;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const bool vis = (R0 + i < M) && (rm >= need);
      const float a = fast_exp2(fmaf(__uint_as_float(v[i]), scale2, -stf[i]));
      hmasked += vis ? a : 0.f;
      if (++rm == m) rm = 0;
    }
  }
}

// CAOTE scores of 256 keys of one unit. grid = (key tile pairs, units), 576 threads: warps 0..15 are the
// key threads, two per key (warps 0..3 and 8..11 the first key tile, 4..7 and 12..15 the second; the
// lower eight take rows 0..63 of every Q block, the upper eight rows 64..127), one lane of warp 16 issues
// the products, one lane of warp 17 the copies.
__global__ void __launch_bounds__(kScoreThreads, 1)
score_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
             const __grid_constant__ CUtensorMap tmV, Dims dm, const int* __restrict__ len, Scratch sc,
             float* __restrict__ scores, int* status) {
  ptx::pdl_wait();
  ptx::pdl_trigger();
  extern __shared__ char smem_raw[];
  // (aligned by an offset into the array, not through an integer: the pointer keeps its address space, and what is
  // read and written through it compiles to shared-memory accesses, not generic ones)
  char* sm = smem_raw + ((1024u - (ptx::smem_u32(smem_raw) & 1023u)) & 1023u);
  char* Ks = sm;                                                     // [2] key tiles
  char* Qst = Ks + 2 * kTileBytes;                                   // [kQStages] Q blocks
  float* Sst = reinterpret_cast<float*>(Qst + kQStages * kTileBytes);  // [kSStages][kTile] row statistics
  float* Xs = Sst + kSStages * kTile;                                // [kD]
  float* hx = Xs + kD;                                               // [kScoreKeys] upper halves' sums
  uint64_t* bars = reinterpret_cast<uint64_t*>(hx + kScoreKeys);
  uint64_t *k_bar = &bars[0], *v_bar = &bars[1], *q_bar = &bars[2], *q_done = q_bar + kQStages, *st_bar = q_done + kQStages,
           *s_bar = st_bar + kSStages, *c_bar = s_bar + 2, *st_free = c_bar + 2;
  constexpr int kBars1 = 2 + 2 * kQStages + kSStages + 2;  // single arrivals (a copy's bytes, a commit)
  constexpr int kBars = kBars1 + 2 + kSStages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + kBars);

  const int tid = threadIdx.x, warp = tid >> 5;
  const int unit = blockIdx.y, j0 = blockIdx.x * kScoreKeys;
  const int b = unit / dm.Hkv;
  const int n = len[b], M = dm.R, m = dm.m;
  if (n == 0 || n < m || n > dm.cap || j0 >= n) return;
  const int nblocks = (M + kTile - 1) / kTile;

  if (tid == 0) {
    for (int i = 0; i < kBars1; ++i) mbar_init(&bars[i], 1);
    for (int i = 0; i < 2; ++i) mbar_init(&c_bar[i], kKeyThreads / 32);  // one arrival per key warp
    for (int i = 0; i < kSStages; ++i) mbar_init(&st_free[i], kKeyThreads / 32);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(tmem_slot, 512);
  if (tid < kD) Xs[tid] = sc.X[(size_t)unit * kD + tid];
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;  // key tile kk, buffer buf: columns [kk * 256 + buf * 128, + 128)
  float h = 0.f;
  const int j = j0 + (tid & (kScoreKeys - 1));  // key threads: this thread's key
  const int rhalf = tid >> 8;                   // key threads: which 64 rows of a Q block

  if (warp == 17) {
    // =============================== copies (one lane) ===============================
    if (tid == kKeyThreads + 32) {
      mbar_expect_tx(k_bar, 2 * kTileBytes);
      for (int kk = 0; kk < 2; ++kk) {
        tma_load_2d(Ks + kk * kTileBytes, &tmK, 0, unit * dm.cap + j0 + kk * kTile, k_bar);
        tma_load_2d(Ks + kk * kTileBytes + kHalfBytes, &tmK, 64, unit * dm.cap + j0 + kk * kTile, k_bar);
      }
      for (int rb = 0; rb < nblocks; ++rb) {
        const int st = rb % kQStages, ss = rb % kSStages;
        if (rb >= kQStages) mbar_wait_idle(&q_done[st], ((rb / kQStages) - 1) & 1, status);  // the products of block rb - 4 are done
        char* qd = Qst + st * kTileBytes;
        mbar_expect_tx(&q_bar[st], kTileBytes);
        tma_load_2d(qd, &tmQ, 0, unit * M + rb * kTile, &q_bar[st]);
        tma_load_2d(qd + kHalfBytes, &tmQ, 64, unit * M + rb * kTile, &q_bar[st]);
        if (rb >= kSStages) mbar_wait_idle(&st_free[ss], ((rb / kSStages) - 1) & 1, status);  // block rb - 8 is summed
        mbar_expect_tx(&st_bar[ss], kStatBytes);
        bulk_load(Sst + ss * kTile, sc.stats + (size_t)unit * sc.Mpad + (size_t)rb * kTile, kStatBytes, &st_bar[ss]);
      }
      // the value rows of the CTA's keys, for the distances at the end: into the first two Q stages once the last
      // product has read its Q block (a commit covers every product before it)
      mbar_wait_idle(&q_done[(nblocks - 1) % kQStages], ((nblocks - 1) / kQStages) & 1, status);
      mbar_expect_tx(v_bar, 2 * kTileBytes);
      for (int kk = 0; kk < 2; ++kk) {
        tma_load_2d(Qst + kk * kTileBytes, &tmV, 0, unit * dm.cap + j0 + kk * kTile, v_bar);
        tma_load_2d(Qst + kk * kTileBytes + kHalfBytes, &tmV, 64, unit * dm.cap + j0 + kk * kTile, v_bar);
      }
    }
  } else if (warp == 16) {
    // =============================== products (one lane) ===============================
    if (tid == kKeyThreads) {
      constexpr uint32_t kIdesc = instr_desc(false);
      const uint32_t k_addr = smem_u32(Ks);
      mbar_wait_idle(k_bar, 0, status);
      for (int rb = 0; rb < nblocks; ++rb) {
        const int buf = rb & 1, st = rb % kQStages;
        mbar_wait_idle(&q_bar[st], (rb / kQStages) & 1, status);
        if (rb >= 2) mbar_wait_idle(&c_bar[buf], ((rb - 2) >> 1) & 1, status);  // its S buffers have been read
        tc_fence_after();
        const uint32_t q_addr = smem_u32(Qst + st * kTileBytes);
#pragma unroll
        for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            umma(tmem + kk * 256 + buf * 128, desc_k_major(k_addr + kk * kTileBytes, ks), desc_k_major(q_addr, ks), kIdesc, ks > 0);
        }
        umma_commit(&s_bar[buf]);
        umma_commit(&q_done[st]);
      }
      // (no arrival may still be on its way to this CTA's barriers when the CTA ends)
      if (nblocks > 0) mbar_wait_idle(&q_done[(nblocks - 1) % kQStages], ((nblocks - 1) / kQStages) & 1, status);
    }
  } else {
    // =============================== one key per thread ===============================
    // A thread's 64 rows of a Q block go through registers in four pieces of 16. Two register sets take turns: while
    // one piece is summed, the next piece's logits (TMEM) and statistics (shared memory) are already on their way, so
    // neither latency is waited for. The S buffer is handed back to the products as soon as its last piece is in
    // registers, not when it has been summed.
    const float scale2 = dm.scale * 1.4426950408889634f;
    const int kk = (warp >> 2) & 1;
    const uint32_t t_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16) + kk * 256 + rhalf * 64;
    const int lane = tid & 31;
    const int need = j - (n - m);  // row R sees key j iff (R % m) >= need
    uint32_t va[16], vb[16];
    float4 sa[4], sb[4];
    float2 hacc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
    mbar_wait(&s_bar[0], 0, status);
    mbar_wait(&st_bar[0], 0, status);
    tc_fence_after();
    tmem_ld16_issue(t_lane, va);
    lds16_issue(Sst + rhalf * 64, sa);
    for (int rb = 0; rb < nblocks; ++rb) {
      const int buf = rb & 1, ss = rb % kSStages;
      // only the keys of the new block itself are masked (causal inside the block), and only the last
      // row block can have columns beyond M
      const bool plain = (j0 + kScoreKeys - 1 < n - m + 1) && (rb * kTile + kTile <= M);
      const int R0 = rb * kTile + rhalf * 64;
      const uint32_t t_s = t_lane + buf * 128;
      const float* stc = Sst + ss * kTile + rhalf * 64;
      // piece 0 (in va / sa); piece 1 on its way
      tmem_ld16_wait(va);
      tmem_ld16_issue(t_s + 16, vb);
      lds16_issue(stc + 16, sb);
      score_piece16(va, sa, scale2, plain, R0, M, m, need, hacc, h);
      // piece 1; piece 2 on its way
      tmem_ld16_wait(vb);
      tmem_ld16_issue(t_s + 32, va);
      lds16_issue(stc + 32, sa);
      score_piece16(vb, sb, scale2, plain, R0 + 16, M, m, need, hacc, h);
      // piece 2; piece 3 on its way
      tmem_ld16_wait(va);
      tmem_ld16_issue(t_s + 48, vb);
      lds16_issue(stc + 48, sb);
      score_piece16(va, sa, scale2, plain, R0 + 32, M, m, need, hacc, h);
      // piece 3; the S buffer is free, the next block's piece 0 on its way
      tmem_ld16_wait(vb);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&c_bar[buf]);  // this warp holds its part of the S buffer in registers
      if (rb + 1 < nblocks) {
        const int ss1 = (rb + 1) % kSStages;
        mbar_wait(&s_bar[buf ^ 1], ((rb + 1) >> 1) & 1, status);
        mbar_wait(&st_bar[ss1], ((rb + 1) / kSStages) & 1, status);  // the next block's row statistics have landed
        tc_fence_after();
        tmem_ld16_issue(t_lane + (buf ^ 1) * 128, va);
        lds16_issue(Sst + ss1 * kTile + rhalf * 64, sa);
      }
      score_piece16(vb, sb, scale2, plain, R0 + 48, M, m, need, hacc, h);
      __syncwarp();
      if (lane == 0) mbar_arrive(&st_free[ss]);  // ... and is done with the block's statistics
    }
    h += (hacc[0].x + hacc[0].y) + (hacc[1].x + hacc[1].y);
  }

  // ---- the two halves of a key add up; then c_j = w_j / (1 - w_j) * ||X - v_j||, w_j = h_j / M ----
  if (tid >= kScoreKeys && tid < kKeyThreads) hx[tid - kScoreKeys] = h;
  __syncthreads();
  if (tid < kScoreKeys) h += hx[tid];
  if (tid < kScoreKeys) mbar_wait(v_bar, 0, status);
  if (tid < kScoreKeys && j < n) {
    // the key's value row: 16 chunks of 8 channels in the staged tile (two boxes of 64 channels, 128-byte swizzle)
    const char* vt = Qst + (tid >> 7) * kTileBytes;
    float acc = 0.f;
#pragma unroll
    for (int c = 0; c < 16; ++c) {
      const uint4 raw = *reinterpret_cast<const uint4*>(vt + tile_off(tid & (kTile - 1), c));
      const uint32_t w4[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const float d0 = Xs[8 * c + 2 * e] - __uint_as_float(w4[e] << 16);
        const float d1 = Xs[8 * c + 2 * e + 1] - __uint_as_float(w4[e] & 0xffff0000u);
        acc = fmaf(d0, d0, acc);
        acc = fmaf(d1, d1, acc);
      }
    }
    const float Htot = (float)M;
    const float rest = Htot - h;
    const float ratio = (rest > 0.f) ? h / rest : INFINITY;
    scores[(size_t)unit * dm.cap + j] = (ratio == 0.f) ? 0.f : ((ratio == INFINITY) ? INFINITY : ratio * sqrtf(acc));
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) tmem_dealloc(tmem, 512);
}

}  // namespace prefill
}  // namespace caote
