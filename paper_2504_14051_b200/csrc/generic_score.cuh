// Generic scoring path: any I/O dtype (bf16 / fp32), head_dim 64 or 128, any block size m, any group
// size up to 16. Plain fp32 CUDA-core arithmetic, three launches:
//
//   attn_partial  split-KV flash attention over tiles of 16 query rows x 64 keys: per (unit, split,
//                 row) running max, running sum and un-normalised partial output; row tile 0 also
//                 accumulates sum_j base_j v_j and sum_j base_j for the base modes that carry scores.
//   attn_combine  merges the splits: final (max, 1/sum) per row, attention output o, and per 32-row
//                 chunk the sum of the output rows that define the base score.
//   score_pass    key-major: a CTA owns 64 cached tokens, recomputes their logits against every
//                 counted query row with the same dot-product routine, sums alpha over rows into h_j,
//                 applies the base mode, and writes c_j = w_j/(1-w_j) * ||X - v_j|| once.
//
// X = sum_j w_j v_j is never formed by a pass of its own: because w is a non-negative combination of
// attention rows (plus the carried base score), X = (sum of the counted output rows + sum_j base_j v_j)
// / (number of counted rows + sum_j base_j).
//
// All reductions run in a fixed order, so results are bit-reproducible from run to run.
#pragma once

#include "common.cuh"

namespace caote {
namespace generic {

constexpr int kRT = 16;          // query rows per tile
constexpr int kKT = 64;          // keys per tile
constexpr int kThreads = 256;
constexpr int kCombineRows = 32; // rows per combine CTA

struct Scratch {
  float* part_ml;  // [units][splits][Rpad][2]   (max logit, sum of exp(s - max) over all keys but the first one at the max)
  float* part_o;   // [units][splits][Rpad][D]
  float* part_y;   // [units][splits][D]
  float* part_hb;  // [units][splits]
  float* stats;    // [units][Rpad][4]   (max, 1/sum, (sum without the row's top key) / sum, unused)
  float* osum;     // [units][chunks][D]
  float* ytot;     // [units][D]
  float* hbtot;    // [units]
  int splits, Rpad, chunks;
};

inline int round_up(int x, int a) { return (x + a - 1) / a * a; }

// Number of key splits: enough CTAs to fill the machine a few times over, never more splits than
// there are 2-tile spans in the cache.
inline int choose_splits(const Dims& dm) {
  const int row_tiles = (dm.R + kRT - 1) / kRT;
  const long ctas = (long)dm.units * row_tiles;
  int s = (int)(((long)g_sm_count * 4 + ctas - 1) / ctas);
  const int max_by_cap = (dm.cap + 2 * kKT - 1) / (2 * kKT);
  if (s > max_by_cap) s = max_by_cap;
  if (s > 32) s = 32;
  if (s < 1) s = 1;
  return s;
}

inline size_t carve(const Dims& dm, char* base, Scratch* out) {
  Scratch s;
  s.splits = choose_splits(dm);
  s.Rpad = round_up(dm.R, kRT);
  s.chunks = (dm.R + kCombineRows - 1) / kCombineRows;
  size_t off = 0;
  auto take = [&](size_t n_floats) {
    float* p = reinterpret_cast<float*>(base + off);
    off = align_up(off + n_floats * sizeof(float), 256);
    return p;
  };
  const size_t us = (size_t)dm.units * s.splits;
  s.part_ml = take(us * s.Rpad * 2);
  s.part_o = take(us * s.Rpad * dm.D);
  s.part_y = take(us * dm.D);
  s.part_hb = take(us);
  s.stats = take((size_t)dm.units * s.Rpad * 4);
  s.osum = take((size_t)dm.units * s.chunks * dm.D);
  s.ytot = take((size_t)dm.units * dm.D);
  s.hbtot = take((size_t)dm.units);
  if (out) *out = s;
  return off;
}

// scale * <q, k> over D channels, in one fixed order, from two fp32 rows in shared memory. Both the
// attention pass and the score pass call this, so a logit has the same bits in both.
template <int D>
__device__ __forceinline__ float logit(const float* __restrict__ qrow, const float* __restrict__ krow,
                                       float scale) {
  float acc = 0.f;
#pragma unroll 8
  for (int c = 0; c < D; c += 4) {
    const float4 a = *reinterpret_cast<const float4*>(qrow + c);
    const float4 b = *reinterpret_cast<const float4*>(krow + c);
    acc = fmaf(a.x, b.x, acc);
    acc = fmaf(a.y, b.y, acc);
    acc = fmaf(a.z, b.z, acc);
    acc = fmaf(a.w, b.w, acc);
  }
  return acc * scale;
}

// Stage `rows` rows of D elements (global, dtype T) into shared memory as fp32 with row stride LD;
// rows at or beyond `valid_rows` are zero-filled.
template <typename T, int D, int LD>
__device__ __forceinline__ void stage_rows(float* dst, const T* src, int rows, int valid_rows) {
  constexpr int V4 = D / 4;
  for (int idx = threadIdx.x; idx < rows * V4; idx += blockDim.x) {
    const int r = idx / V4, c4 = idx % V4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < valid_rows) v = load4(src + (size_t)r * D + c4 * 4);
    *reinterpret_cast<float4*>(dst + r * LD + c4 * 4) = v;
  }
}

// Row r of a unit: query head g = r / m, query i = r % m.
__device__ __forceinline__ size_t q_offset(const Dims& dm, int b, int h, int r) {
  const int g = r / dm.m, i = r % dm.m;
  return (((size_t)b * dm.Hq + h * dm.G + g) * dm.m + i) * dm.D;
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
attn_partial_kernel(Dims dm, const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                    const int* __restrict__ len, const float* __restrict__ base, Scratch sc, int* status) {
  constexpr int LD = D + 4;
  constexpr int OC = D / 16;  // output channels per thread (two float4 for D = 128, one for D = 64)
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Ks = Qs + kRT * LD;
  float* Vs = Ks + kKT * LD;
  float* Ps = Vs + kKT * LD;
  float* bs = Ps + kRT * kKT;   // kKT base values
  float* red = bs + kKT;        // kThreads floats

  const int unit = blockIdx.z, split = blockIdx.y, rt = blockIdx.x;
  const int b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b];
  if (threadIdx.x == 0 && unit == 0 && split == 0 && rt == 0) status[kStatTagIndex] = kStatNone;
  if (n == 0) return;
  if (n < dm.m || n > dm.cap) {
    if (threadIdx.x == 0) set_status(status, CAOTE_ERR_BAD_LENGTH);
    return;
  }
  const bool use_base = (dm.base_mode == CAOTE_BASE_ACCUM || dm.base_mode == CAOTE_BASE_EXTERNAL) && rt == 0;
  const int tid = threadIdx.x, r = tid >> 4, c0 = tid & 15;
  const int r_glob = rt * kRT + r;
  const bool row_ok = r_glob < dm.R;
  const int n_vis = row_ok ? n - dm.m + (r_glob % dm.m) + 1 : 0;

  // stage the query tile
  for (int idx = tid; idx < kRT * (D / 4); idx += kThreads) {
    const int rr = idx / (D / 4), c4 = idx % (D / 4);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (rt * kRT + rr < dm.R) v = load4(q + q_offset(dm, b, h, rt * kRT + rr) + c4 * 4);
    *reinterpret_cast<float4*>(Qs + rr * LD + c4 * 4) = v;
  }

  const int split_len = ((n + sc.splits - 1) / sc.splits + kKT - 1) / kKT * kKT;
  const int k_begin = split * split_len;
  const int k_end = min(n, k_begin + split_len);
  const T* Ku = K + (size_t)unit * dm.cap * D;
  const T* Vu = V + (size_t)unit * dm.cap * D;

  // l_rest: sum of exp(s - m_run) over the keys so far EXCEPT the first key that sits at the maximum (whose
  // term is exactly 1): the row's 1 - alpha of its top key is then l_rest / (l_rest + 1), a sum of the others
  float m_run = -INFINITY, l_rest = 0.f;
  float o_acc[OC];
#pragma unroll
  for (int i = 0; i < OC; ++i) o_acc[i] = 0.f;
  float y_acc = 0.f, hb_acc = 0.f;
  constexpr int YP = kThreads / D;  // threads per channel in the base-weighted value sum

  for (int kt = k_begin; kt < k_end; kt += kKT) {
    __syncthreads();
    stage_rows<T, D, LD>(Ks, Ku + (size_t)kt * D, kKT, k_end - kt);
    stage_rows<T, D, LD>(Vs, Vu + (size_t)kt * D, kKT, k_end - kt);
    if (use_base && tid < kKT) bs[tid] = (kt + tid < k_end) ? base[(size_t)unit * dm.cap + kt + tid] : 0.f;
    __syncthreads();

    float s[4];
    float mx = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int j = kt + c0 + 16 * i;
      s[i] = (j < k_end && j < n_vis) ? logit<D>(Qs + r * LD, Ks + (c0 + 16 * i) * LD, dm.scale) : -INFINITY;
      mx = fmaxf(mx, s[i]);
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float m_new = fmaxf(m_run, mx);
    const bool new_top = mx > m_run;  // this tile holds a key above everything before it
    // (no branch here: the two rows of a warp vote together below)
    const float corr = (m_run == -INFINITY) ? 0.f : expf(m_run - m_new);
    float lsum = 0.f;
    bool found = false;  // the first key of the tile at the new maximum (smallest key index) is left out of the sum
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float p = (s[i] == -INFINITY) ? 0.f : expf(s[i] - m_new);
      Ps[r * kKT + c0 + 16 * i] = p;
      const unsigned at_top = (__ballot_sync(0xffffffffu, new_top && s[i] == m_new) >> (threadIdx.x & 16)) & 0xffffu;
      const bool skip = !found && at_top != 0u && (int)(__ffs(at_top) - 1) == c0;
      found |= at_top != 0u;
      lsum += skip ? 0.f : p;
    }
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, o);
    // the old top key (term 1 before) joins the others when a new top appears
    l_rest = l_rest * corr + ((new_top && m_run != -INFINITY) ? corr : 0.f) + lsum;
    m_run = m_new;
#pragma unroll
    for (int i = 0; i < OC; ++i) o_acc[i] *= corr;
    __syncthreads();

    for (int j = 0; j < kKT; ++j) {
      const float p = Ps[r * kKT + j];
      const float4 v0 = *reinterpret_cast<const float4*>(Vs + j * LD + c0 * 4);
      o_acc[0] = fmaf(p, v0.x, o_acc[0]);
      o_acc[1] = fmaf(p, v0.y, o_acc[1]);
      o_acc[2] = fmaf(p, v0.z, o_acc[2]);
      o_acc[3] = fmaf(p, v0.w, o_acc[3]);
      if (OC == 8) {
        const float4 v1 = *reinterpret_cast<const float4*>(Vs + j * LD + 64 + c0 * 4);
        o_acc[4] = fmaf(p, v1.x, o_acc[4]);
        o_acc[5] = fmaf(p, v1.y, o_acc[5]);
        o_acc[6] = fmaf(p, v1.z, o_acc[6]);
        o_acc[7] = fmaf(p, v1.w, o_acc[7]);
      }
    }
    if (use_base) {
      const int col = tid % D, part = tid / D;
      for (int j = part; j < kKT; j += YP) y_acc = fmaf(bs[j], Vs[j * LD + col], y_acc);
      if (tid < kKT) hb_acc += bs[tid];
    }
  }

  const size_t us = (size_t)unit * sc.splits + split;
  if (row_ok) {
    if (c0 == 0) {
      sc.part_ml[(us * sc.Rpad + r_glob) * 2 + 0] = m_run;
      sc.part_ml[(us * sc.Rpad + r_glob) * 2 + 1] = l_rest;
    }
    float* po = sc.part_o + (us * sc.Rpad + r_glob) * D;
    *reinterpret_cast<float4*>(po + c0 * 4) = make_float4(o_acc[0], o_acc[1], o_acc[2], o_acc[3]);
    if (OC == 8)
      *reinterpret_cast<float4*>(po + 64 + c0 * 4) = make_float4(o_acc[4], o_acc[5], o_acc[6], o_acc[7]);
  }
  if (use_base) {
    __syncthreads();
    red[tid] = y_acc;
    __syncthreads();
    if (tid < D) {
      float y = 0.f;
      for (int p = 0; p < YP; ++p) y += red[p * D + tid];
      sc.part_y[us * D + tid] = y;
    }
    __syncthreads();
    red[tid] = (tid < kKT) ? hb_acc : 0.f;
    __syncthreads();
    if (tid == 0) {
      float hsum = 0.f;
      for (int j = 0; j < kKT; ++j) hsum += red[j];
      sc.part_hb[us] = hsum;
    }
  }
}

// Is row r one of the rows whose attention defines the base score?
__device__ __forceinline__ bool row_counted(const Dims& dm, int r) {
  if (dm.base_mode == CAOTE_BASE_LAST_QUERY) return (r % dm.m) == dm.m - 1;
  return dm.base_mode != CAOTE_BASE_EXTERNAL;
}

template <typename T, int D>
__global__ void __launch_bounds__(D)
attn_combine_kernel(Dims dm, const int* __restrict__ len, Scratch sc, float* __restrict__ o) {
  const int unit = blockIdx.y, chunk = blockIdx.x, c = threadIdx.x;
  const int b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b];
  if (n == 0 || n < dm.m || n > dm.cap) return;
  float osum = 0.f;
  const int r_end = min(dm.R, (chunk + 1) * kCombineRows);
  for (int r = chunk * kCombineRows; r < r_end; ++r) {
    float mx = -INFINITY;
    for (int s = 0; s < sc.splits; ++s)
      mx = fmaxf(mx, sc.part_ml[(((size_t)unit * sc.splits + s) * sc.Rpad + r) * 2]);
    float l_rest = 0.f, acc = 0.f;
    bool top_seen = false;  // the first split at the overall maximum keeps its top key apart; the others' join the rest
    for (int s = 0; s < sc.splits; ++s) {
      const size_t idx = ((size_t)unit * sc.splits + s) * sc.Rpad + r;
      const float ms = sc.part_ml[idx * 2];
      if (ms == -INFINITY) continue;
      const float f = expf(ms - mx);
      l_rest = fmaf(sc.part_ml[idx * 2 + 1], f, l_rest);
      if (ms == mx && !top_seen) top_seen = true;
      else l_rest += f;
      acc = fmaf(sc.part_o[idx * D + c], f, acc);
    }
    const float inv_l = 1.f / (l_rest + 1.f);
    const float val = acc * inv_l;
    o[q_offset(dm, b, h, r) + c] = val;
    if (row_counted(dm, r)) osum += val;
    if (c == 0) {
      sc.stats[((size_t)unit * sc.Rpad + r) * 4 + 0] = mx;
      sc.stats[((size_t)unit * sc.Rpad + r) * 4 + 1] = inv_l;
      sc.stats[((size_t)unit * sc.Rpad + r) * 4 + 2] = l_rest * inv_l;
    }
  }
  sc.osum[((size_t)unit * sc.chunks + chunk) * D + c] = osum;
  if (chunk == 0 && (dm.base_mode == CAOTE_BASE_ACCUM || dm.base_mode == CAOTE_BASE_EXTERNAL)) {
    float y = 0.f;
    for (int s = 0; s < sc.splits; ++s) y += sc.part_y[((size_t)unit * sc.splits + s) * D + c];
    sc.ytot[(size_t)unit * D + c] = y;
    if (c == 0) {
      double hb = 0.0;
      for (int s = 0; s < sc.splits; ++s) hb += (double)sc.part_hb[(size_t)unit * sc.splits + s];
      sc.hbtot[unit] = (float)hb;
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
score_pass_kernel(Dims dm, const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                  const int* __restrict__ len, float* __restrict__ base, Scratch sc,
                  float* __restrict__ scores, const float* __restrict__ vsum) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;              // kRT * LD
  float* Ks = Qs + kRT * LD;     // kKT * LD
  float* Hred = Ks + kKT * LD;   // kRT * kKT  sums of the rows' weights of a key
  float* Cred = Hred + kRT * kKT;  // kRT * kKT  sums of the rows' complements 1 - alpha of a key
  float* Xs = Cred + kRT * kKT;  // D
  float* st = Xs + D;            // kRT * 4
  float* wq = st + kRT * 4;      // kKT: w_j / (1 - w_j)

  const int unit = blockIdx.y;
  const int b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b];
  const int j0 = blockIdx.x * kKT;
  if (n == 0 || n < dm.m || n > dm.cap || j0 >= n) return;
  const int tid = threadIdx.x, r = tid >> 4, c0 = tid & 15;
  const int mode = dm.base_mode;
  const int n_rows = (mode == CAOTE_BASE_LAST_QUERY) ? dm.G : (mode == CAOTE_BASE_EXTERNAL ? 0 : dm.R);
  const bool carried = (mode == CAOTE_BASE_ACCUM || mode == CAOTE_BASE_EXTERNAL);
  const float hb = carried ? sc.hbtot[unit] : 0.f;
  const float Htot = (float)n_rows + hb;

  // X = (sum of counted output rows + sum_j base_j v_j) / (counted rows + sum_j base_j)
  if (tid < D) {
    float x = 0.f;
    for (int ch = 0; ch < sc.chunks; ++ch) x += sc.osum[((size_t)unit * sc.chunks + ch) * D + tid];
    if (carried) x += sc.ytot[(size_t)unit * D + tid];
    Xs[tid] = (Htot > 0.f) ? x / Htot : 0.f;
    if (vsum) Xs[tid] = vsum[(size_t)unit * D + tid] / (float)n;  // FastCAOTE (Sec. 3.3): the mean of the cached values
  }
  const int valid = min(kKT, n - j0);
  if (n_rows > 0) stage_rows<T, D, LD>(Ks, K + ((size_t)unit * dm.cap + j0) * D, kKT, valid);

  // hacc: sum over the counted rows of alpha_{r,j}; cacc: sum of 1 - alpha_{r,j}, where the row's top key takes
  // (sum of the others) / sum from the attention pass and everybody else 1 - alpha <= 1/2: no cancellation
  float hacc[4] = {0.f, 0.f, 0.f, 0.f}, cacc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int t0 = 0; t0 < n_rows; t0 += kRT) {
    __syncthreads();
    // counted row number t -> row of the unit
    for (int idx = tid; idx < kRT * (D / 4); idx += kThreads) {
      const int rr = idx / (D / 4), c4 = idx % (D / 4);
      const int t = t0 + rr;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (t < n_rows) {
        const int row = (mode == CAOTE_BASE_LAST_QUERY) ? t * dm.m + dm.m - 1 : t;
        v = load4(q + q_offset(dm, b, h, row) + c4 * 4);
      }
      *reinterpret_cast<float4*>(Qs + rr * LD + c4 * 4) = v;
    }
    if (tid < kRT) {
      const int t = t0 + tid;
      float mx = 0.f, il = 0.f, cr = 0.f;
      if (t < n_rows) {
        const int row = (mode == CAOTE_BASE_LAST_QUERY) ? t * dm.m + dm.m - 1 : t;
        mx = sc.stats[((size_t)unit * sc.Rpad + row) * 4];
        il = sc.stats[((size_t)unit * sc.Rpad + row) * 4 + 1];
        cr = sc.stats[((size_t)unit * sc.Rpad + row) * 4 + 2];
      }
      st[tid * 4] = mx;
      st[tid * 4 + 1] = il;
      st[tid * 4 + 2] = cr;
    }
    __syncthreads();
    const int t = t0 + r;
    if (t < n_rows) {
      const int row = (mode == CAOTE_BASE_LAST_QUERY) ? t * dm.m + dm.m - 1 : t;
      const int n_vis = n - dm.m + (row % dm.m) + 1;
      const float mx = st[r * 4], il = st[r * 4 + 1], cr = st[r * 4 + 2];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int j = j0 + c0 + 16 * i;
        if (j < n_vis) {
          const float sl = logit<D>(Qs + r * LD, Ks + (c0 + 16 * i) * LD, dm.scale);
          const float a = expf(sl - mx) * il;
          hacc[i] += a;
          cacc[i] += (sl == mx) ? cr : 1.f - a;
        } else {
          cacc[i] += 1.f;  // a row that cannot see the key gives all its weight to the others
        }
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    Hred[r * kKT + c0 + 16 * i] = hacc[i];
    Cred[r * kKT + c0 + 16 * i] = cacc[i];
  }
  __syncthreads();
  if (tid < kKT) {
    const int j = j0 + tid;
    float ratio = 0.f;
    if (j < n) {
      float hj = 0.f, rest = 0.f;  // rest = (1 - w_j) * Htot as a sum of non-negative parts
      for (int rr = 0; rr < kRT; ++rr) {
        hj += Hred[rr * kKT + tid];
        rest += Cred[rr * kKT + tid];
      }
      if (carried) {
        // (the carried scores' own complement is a plain difference: a single carried score that holds almost
        // all of their sum is outside what this any-shape path resolves)
        const float bj = base[(size_t)unit * dm.cap + j];
        rest += hb - bj;
        if (mode == CAOTE_BASE_ACCUM) {
          hj += bj;
          base[(size_t)unit * dm.cap + j] = hj;
        } else {
          hj = bj;
        }
      }
      if (Htot > 0.f && hj > 0.f) ratio = (rest > 0.f) ? hj / rest : INFINITY;
    }
    wq[tid] = ratio;
  }
  __syncthreads();
  // || X - v_j ||: 4 threads per token, D/4 consecutive channels each
  {
    const int key = tid >> 2, part = tid & 3;
    const int j = j0 + key;
    float acc = 0.f;
    if (j < n) {
      const T* vrow = V + ((size_t)unit * dm.cap + j) * D + part * (D / 4);
#pragma unroll
      for (int c = 0; c < D / 4; c += 4) {
        const float4 v = load4(vrow + c);
        const float* x = Xs + part * (D / 4) + c;
        const float d0 = x[0] - v.x, d1 = x[1] - v.y, d2 = x[2] - v.z, d3 = x[3] - v.w;
        acc = fmaf(d0, d0, acc);
        acc = fmaf(d1, d1, acc);
        acc = fmaf(d2, d2, acc);
        acc = fmaf(d3, d3, acc);
      }
    }
    acc += __shfl_xor_sync(0xffffffffu, acc, 1);
    acc += __shfl_xor_sync(0xffffffffu, acc, 2);
    if (part == 0 && j < n) {
      const float ratio = wq[key];
      const float nrm = sqrtf(acc);
      // ratio == +inf with a zero distance still means "holds all the weight": keep +inf
      scores[(size_t)unit * dm.cap + j] = (ratio == 0.f) ? 0.f : ((ratio == INFINITY) ? INFINITY : ratio * nrm);
    }
  }
}

inline size_t partial_smem(int D) {
  const int LD = D + 4;
  return sizeof(float) * (size_t)(kRT * LD + 2 * kKT * LD + kRT * kKT + kKT + kThreads);
}
// Sum-of-errors aggregation: instead of adding the rows' weights and applying the general form once,
// add up the exact single-query errors (Theorem 3.2, row by row) of the rows that define the base score:
//     c_j = sum_r alpha_{r,j} / (1 - alpha_{r,j}) * || o_r - v_j ||_2 .
// Needs o and the row statistics of attn_partial / attn_combine. grid = (key tiles, units), kThreads;
// thread (r = tid / 16, c0 = tid % 16) owns row slot r and keys c0 + 16 i of the tile.
template <typename T, int D>
__global__ void __launch_bounds__(kThreads)
sum_errors_kernel(Dims dm, const T* __restrict__ q, const T* __restrict__ K, const T* __restrict__ V,
                  const int* __restrict__ len, const float* __restrict__ o, Scratch sc, float* __restrict__ scores) {
  constexpr int LD = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;              // kRT * LD
  float* Os = Qs + kRT * LD;     // kRT * LD
  float* Ks = Os + kRT * LD;     // kKT * LD
  float* Vs = Ks + kKT * LD;     // kKT * LD
  float* Hred = Vs + kKT * LD;   // kRT * kKT
  float* st = Hred + kRT * kKT;  // kRT * 2

  const int unit = blockIdx.y;
  const int b = unit / dm.Hkv, h = unit % dm.Hkv;
  const int n = len[b];
  const int j0 = blockIdx.x * kKT;
  if (n == 0 || n < dm.m || n > dm.cap || j0 >= n) return;
  const int tid = threadIdx.x, r = tid >> 4, c0 = tid & 15;
  const int mode = dm.base_mode;
  const int n_rows = (mode == CAOTE_BASE_LAST_QUERY) ? dm.G : dm.R;
  const int valid = min(kKT, n - j0);
  stage_rows<T, D, LD>(Ks, K + ((size_t)unit * dm.cap + j0) * D, kKT, valid);
  stage_rows<T, D, LD>(Vs, V + ((size_t)unit * dm.cap + j0) * D, kKT, valid);

  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int t0 = 0; t0 < n_rows; t0 += kRT) {
    __syncthreads();
    for (int idx = tid; idx < kRT * (D / 4); idx += kThreads) {
      const int rr = idx / (D / 4), c4 = idx % (D / 4);
      const int t = t0 + rr;
      float4 qv = make_float4(0.f, 0.f, 0.f, 0.f), ov = qv;
      if (t < n_rows) {
        const int row = (mode == CAOTE_BASE_LAST_QUERY) ? t * dm.m + dm.m - 1 : t;
        qv = load4(q + q_offset(dm, b, h, row) + c4 * 4);
        ov = *reinterpret_cast<const float4*>(o + q_offset(dm, b, h, row) + c4 * 4);
      }
      *reinterpret_cast<float4*>(Qs + rr * LD + c4 * 4) = qv;
      *reinterpret_cast<float4*>(Os + rr * LD + c4 * 4) = ov;
    }
    if (tid < kRT) {
      const int t = t0 + tid;
      float mx = 0.f, il = 0.f, cr = 0.f;
      if (t < n_rows) {
        const int row = (mode == CAOTE_BASE_LAST_QUERY) ? t * dm.m + dm.m - 1 : t;
        mx = sc.stats[((size_t)unit * sc.Rpad + row) * 4];
        il = sc.stats[((size_t)unit * sc.Rpad + row) * 4 + 1];
        cr = sc.stats[((size_t)unit * sc.Rpad + row) * 4 + 2];
      }
      st[tid * 4] = mx;
      st[tid * 4 + 1] = il;
      st[tid * 4 + 2] = cr;
    }
    __syncthreads();
    const int t = t0 + r;
    if (t < n_rows) {
      const int row = (mode == CAOTE_BASE_LAST_QUERY) ? t * dm.m + dm.m - 1 : t;
      const int n_vis = n - dm.m + (row % dm.m) + 1;
      const float mx = st[r * 4], il = st[r * 4 + 1], cr = st[r * 4 + 2];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int jj = c0 + 16 * i, j = j0 + jj;
        if (j < n_vis) {
          const float sl = logit<D>(Qs + r * LD, Ks + jj * LD, dm.scale);
          const float e = expf(sl - mx) * il;              // alpha
          const float rest = (sl == mx) ? cr : 1.f - e;    // 1 - alpha: the others' share, without cancellation
          float d2 = 0.f;
#pragma unroll 8
          for (int c = 0; c < D; c += 4) {
            const float4 ov = *reinterpret_cast<const float4*>(Os + r * LD + c);
            const float4 vv = *reinterpret_cast<const float4*>(Vs + jj * LD + c);
            const float a0 = ov.x - vv.x, a1 = ov.y - vv.y, a2 = ov.z - vv.z, a3 = ov.w - vv.w;
            d2 = fmaf(a0, a0, d2); d2 = fmaf(a1, a1, d2); d2 = fmaf(a2, a2, d2); d2 = fmaf(a3, a3, d2);
          }
          acc[i] += (rest > 0.f) ? e / rest * sqrtf(d2) : INFINITY;
        }
      }
    }
  }
  __syncthreads();
#pragma unroll
  for (int i = 0; i < 4; ++i) Hred[r * kKT + c0 + 16 * i] = acc[i];
  __syncthreads();
  if (tid < kKT && j0 + tid < n) {
    float cj = 0.f;
    for (int rr = 0; rr < kRT; ++rr) cj += Hred[rr * kKT + tid];
    scores[(size_t)unit * dm.cap + j0 + tid] = cj;
  }
}

inline size_t sum_errors_smem(int D) {
  const int LD = D + 4;
  return sizeof(float) * (size_t)(2 * kRT * LD + 2 * kKT * LD + kRT * kKT + kRT * 4);
}

inline size_t score_smem(int D) {
  const int LD = D + 4;
  return sizeof(float) * (size_t)(kRT * LD + kKT * LD + 2 * kRT * kKT + D + kRT * 4 + kKT);
}

}  // namespace generic
}  // namespace caote
