// C ABI of the CAOTE library: argument validation, workspace carving and kernel dispatch.
// Every entry point only enqueues work on the caller's stream.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <utility>
#include <vector>

#include "common.cuh"
#include "decode_cluster.cuh"
#include "decode_tc.cuh"
#include "generic_score.cuh"
#include "greedy.cuh"
#include "greedy_cluster.cuh"
#include "post_evict.cuh"
#include "prefill_tc.cuh"
#include "select_compact.cuh"
#include "sum_errors_decode.cuh"

namespace caote {

static std::atomic<long long> g_launches{0};
static std::atomic<long long> g_wait_cycles{2000000000LL};  // CAOTE_OPT_WAIT_CYCLES
static std::atomic<int> g_side_by_side{1};                  // CAOTE_OPT_SIDE_BY_SIDE: 0 off, 1 when it pays
static std::atomic<int> g_decode_cluster{0};                // CAOTE_OPT_DECODE_CLUSTER: 0 auto, -1 off, else the size
static thread_local char g_cuda_error[256] = "";

static int cuda_fail(cudaError_t e, const char* what) {
  snprintf(g_cuda_error, sizeof(g_cuda_error), "%s: %s", what, cudaGetErrorString(e));
  return CAOTE_ERR_CUDA;
}
#define CAOTE_CUDA(call)                                  \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
  } while (0)

static int after_launch(const char* name) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, name);
  return CAOTE_OK;
}

// ---- optional per-kernel tracing: CUDA events recorded on the launching stream around each kernel ----
struct TraceRec {
  const char* name;
  cudaEvent_t a, b;
};
static std::atomic<bool> g_trace_on{false};
static std::mutex g_trace_mu;
static std::vector<TraceRec> g_trace_pending;
static std::vector<cudaEvent_t> g_trace_pool;

static cudaEvent_t trace_event() {
  std::lock_guard<std::mutex> lk(g_trace_mu);
  if (!g_trace_pool.empty()) {
    cudaEvent_t e = g_trace_pool.back();
    g_trace_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
  return e;
}

struct TraceScope {
  const char* name;
  cudaStream_t st;
  cudaEvent_t a = nullptr, b = nullptr;
  TraceScope(const char* n, cudaStream_t s) : name(n), st(s) {
    if (!g_trace_on.load(std::memory_order_relaxed)) return;
    a = trace_event();
    b = trace_event();
    if (a && b) cudaEventRecord(a, st);
  }
  ~TraceScope() {
    if (!a || !b) return;
    cudaEventRecord(b, st);
    std::lock_guard<std::mutex> lk(g_trace_mu);
    g_trace_pending.push_back({name, a, b});
  }
};

// Launch a kernel (the statement after the stream argument), count it, trace it when tracing is on,
// and return from the calling function if the launch failed.
#define CAOTE_LAUNCH(name, st, ...)        \
  do {                                     \
    int rc__;                              \
    {                                      \
      TraceScope ts__(name, st);           \
      __VA_ARGS__;                         \
      rc__ = after_launch(name);           \
    }                                      \
    if (rc__ != CAOTE_OK) return rc__;     \
  } while (0)

// Launch with the programmatic-serialization attribute: the kernel may be scheduled while its predecessor in the
// stream is still running and waits for it in its first statement (ptx::pdl_wait). Only for kernels that do so.
template <typename... KArgs, typename... Args>
static void launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  (void)cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);  // (errors are picked up by after_launch)
}

static bool params_ok(const caote_params_t* p) {
  if (!p) return false;
  if (p->batch < 1 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->capacity < 1 || p->n_new < 1) return false;
  if (p->n_q_heads % p->n_kv_heads != 0) return false;
  if (p->n_q_heads / p->n_kv_heads > 16) return false;
  if (p->n_new > p->capacity) return false;
  if (p->flags != 0) return false;
  if (p->base_mode < CAOTE_BASE_LAST_QUERY || p->base_mode > CAOTE_BASE_EXTERNAL) return false;
  if (!(p->scale == p->scale)) return false;
  return true;
}
static bool params_supported(const caote_params_t* p) {
  if (p->dtype != CAOTE_BF16 && p->dtype != CAOTE_F32) return false;
  if (p->head_dim != 64 && p->head_dim != 128) return false;
  return true;
}

static Dims make_dims(const caote_params_t* p) {
  Dims d;
  d.B = p->batch;
  d.Hq = p->n_q_heads;
  d.Hkv = p->n_kv_heads;
  d.G = d.Hq / d.Hkv;
  d.D = p->head_dim;
  d.cap = p->capacity;
  d.m = p->n_new;
  d.R = d.G * d.m;
  d.units = d.B * d.Hkv;
  d.scale = p->scale;
  d.base_mode = p->base_mode;
  return d;
}

// The device must be a compute-capability 10.x part; checked once per device.
static int check_device() {
  static std::atomic<int> ok[64];
  int dev = 0;
  CAOTE_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return CAOTE_ERR_UNSUPPORTED;
  int st = ok[dev].load(std::memory_order_acquire);
  if (st == 0) {
    int major = 0;
    CAOTE_CUDA(cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev));
    st = (major == 10) ? 1 : -1;
    ok[dev].store(st, std::memory_order_release);
  }
  return st == 1 ? CAOTE_OK : CAOTE_ERR_UNSUPPORTED;
}

template <typename KernelT>
static int allow_smem(KernelT kernel, size_t bytes) {
  if (bytes > 48 * 1024)
    CAOTE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes));
  return CAOTE_OK;
}

template <typename T, int D>
static int launch_generic_score(const Dims& dm, const void* q, const void* K, const void* V, const int* len,
                                float* base, float* o, float* scores, char* ws, cudaStream_t st, const float* vsum,
                                bool sum_errors = false) {
  generic::Scratch sc;
  generic::carve(dm, ws + kHeaderBytes, &sc);
  int* status = reinterpret_cast<int*>(ws);
  const int row_tiles = (dm.R + generic::kRT - 1) / generic::kRT;
  {
    const size_t smem = generic::partial_smem(D);
    int rc = allow_smem(generic::attn_partial_kernel<T, D>, smem);
    if (rc) return rc;
    dim3 grid(row_tiles, sc.splits, dm.units);
    CAOTE_LAUNCH("attn_partial_kernel", st, generic::attn_partial_kernel<T, D><<<grid, generic::kThreads, smem, st>>>(
        dm, (const T*)q, (const T*)K, (const T*)V, len, base, sc, status));
  }
  {
    dim3 grid(sc.chunks, dm.units);
    CAOTE_LAUNCH("attn_combine_kernel", st, generic::attn_combine_kernel<T, D><<<grid, D, 0, st>>>(dm, len, sc, o));
  }
  if (sum_errors) {
    const size_t smem = generic::sum_errors_smem(D);
    int rc = allow_smem(generic::sum_errors_kernel<T, D>, smem);
    if (rc) return rc;
    dim3 grid((dm.cap + generic::kKT - 1) / generic::kKT, dm.units);
    CAOTE_LAUNCH("sum_errors_kernel", st, generic::sum_errors_kernel<T, D><<<grid, generic::kThreads, smem, st>>>(
        dm, (const T*)q, (const T*)K, (const T*)V, len, o, sc, scores));
    return CAOTE_OK;
  }
  {
    const size_t smem = generic::score_smem(D);
    int rc = allow_smem(generic::score_pass_kernel<T, D>, smem);
    if (rc) return rc;
    dim3 grid((dm.cap + generic::kKT - 1) / generic::kKT, dm.units);
    CAOTE_LAUNCH("score_pass_kernel", st, generic::score_pass_kernel<T, D><<<grid, generic::kThreads, smem, st>>>(
        dm, (const T*)q, (const T*)K, (const T*)V, len, base, sc, scores, vsum));
  }
  return CAOTE_OK;
}

// ---- single-query fast path ---------------------------------------------------------------------
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static TensorMapEncodeFn tensor_map_encoder() {
  static std::atomic<TensorMapEncodeFn> fn{nullptr};
  TensorMapEncodeFn f = fn.load(std::memory_order_acquire);
  if (!f) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qr) == cudaSuccess &&
        qr == cudaDriverEntryPointSuccess)
      f = reinterpret_cast<TensorMapEncodeFn>(ptr);
    fn.store(f, std::memory_order_release);
  }
  return f;
}

// Resident CTAs of the persistent decode kernel on the current device (SMs x CTAs per SM); 0 on error.
static int decode_grid_limit() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int g = cached[dev].load(std::memory_order_acquire);
  if (g == 0) {
    int sms = 0, per_sm = 0;
    const size_t smem = decode::tc_smem_bytes(false);
    const size_t smem_fast = decode::tc_smem_bytes(true);
    if (cudaFuncSetAttribute(decode::decode_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess ||
        cudaFuncSetAttribute(decode::decode_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_fast) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, decode::decode_tc_kernel<false>, decode::kTcThreads, smem) != cudaSuccess)
      return 0;
    g = sms * per_sm;
    cached[dev].store(g > 0 ? g : -1, std::memory_order_release);
  }
  return g > 0 ? g : 0;
}

static inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

// Shapes the persistent decode kernel covers; everything else takes the generic path.
static bool decode_shape_ok(const caote_params_t* p) {
  const int G = p->n_q_heads / p->n_kv_heads;
  const bool carried = p->base_mode == CAOTE_BASE_ACCUM || p->base_mode == CAOTE_BASE_EXTERNAL;
  // a carried base score rides in row 7 of the P operand (G <= 7) and is staged by 16-byte bulk copies
  return p->dtype == CAOTE_BF16 && p->head_dim == 128 && p->n_new == 1 && G <= 8 &&
         !(carried && (G > 7 || p->capacity % 4 != 0)) &&
         (long long)p->batch * p->n_kv_heads * p->capacity < (1LL << 31);
}

// ---- single-query path on thread-block clusters ---------------------------------------------------------
typedef void (*ClusterKernel)(const CUtensorMap, const CUtensorMap, const CUtensorMap, Dims, const int*, float*, float*,
                              float*, int*, long long, const float*);
template <int kMode>
static ClusterKernel cluster_kernel_for_g(int g) {
  switch (g) {
    case 1: return dcl::decode_cluster_kernel<1, kMode>;
    case 2: return dcl::decode_cluster_kernel<2, kMode>;
    case 3: return dcl::decode_cluster_kernel<3, kMode>;
    case 4: return dcl::decode_cluster_kernel<4, kMode>;
    case 5: return dcl::decode_cluster_kernel<5, kMode>;
    case 6: return dcl::decode_cluster_kernel<6, kMode>;
    case 7: return dcl::decode_cluster_kernel<7, kMode>;
    default: return dcl::decode_cluster_kernel<8, kMode>;
  }
}
// The instantiation for a group size and a base mode (LAST_QUERY and CHUNK_SUM coincide for one query).
static ClusterKernel cluster_kernel(int g, int base_mode) {
  if (base_mode == CAOTE_BASE_ACCUM) return cluster_kernel_for_g<CAOTE_BASE_ACCUM>(g > 7 ? 7 : g);
  if (base_mode == CAOTE_BASE_EXTERNAL) return cluster_kernel_for_g<CAOTE_BASE_EXTERNAL>(g > 7 ? 7 : g);
  return cluster_kernel_for_g<CAOTE_BASE_LAST_QUERY>(g);
}

// Clusters of `c` CTAs of the cluster kernel that can be resident on the current device at once; 0 if none.
static int cluster_capacity(int c, ClusterKernel kernel) {
  static std::atomic<int> cached[64][dcl::kMaxC + 1];
  int dev = 0;
  if (c < 1 || c > dcl::kMaxC || cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int n = cached[dev][c].load(std::memory_order_acquire);
  if (n == 0) {
    const size_t smem = dcl::smem_bytes();
    n = -1;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess &&
        cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3((unsigned)c * 64u);
      cfg.blockDim = dim3(dcl::kThreads);
      cfg.dynamicSmemBytes = smem;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = (unsigned)c;
      at[0].val.clusterDim.y = 1;
      at[0].val.clusterDim.z = 1;
      cfg.attrs = at;
      cfg.numAttrs = 1;
      int got = 0;
      if (cudaOccupancyMaxActiveClusters(&got, kernel, &cfg) == cudaSuccess && got > 0) n = got;
    }
    (void)cudaGetLastError();
    cached[dev][c].store(n, std::memory_order_release);
  }
  return n > 0 ? n : 0;
}

// Cluster size for these dimensions: every CTA must be able to keep its share of a full unit (kMaxT
// tiles), and among the sizes that can, the one with the smallest estimate of rounds x (tiles per CTA +
// a fixed cost per unit for the merge) wins. 0: no size fits (the unit is too long, or no cluster can run).
static int choose_cluster(const Dims& dm, ClusterKernel kernel, int* clusters_out) {
  const int cap_tiles = (dm.cap + decode::kT - 1) / decode::kT;
  const int forced = g_decode_cluster.load(std::memory_order_relaxed);
  if (forced < 0) return 0;
  int best = 0, best_n = 0;
  double best_cost = 0.0;
  for (int c = 1; c <= dcl::kMaxC; ++c) {
    if (forced > 0 && c != forced) continue;
    if ((cap_tiles + c - 1) / c > dcl::kMaxT) continue;
    const int n = cluster_capacity(c, kernel);
    if (n <= 0) continue;
    const long long rounds = ((long long)dm.units + n - 1) / n;
    const double cost = (double)rounds * ((double)cap_tiles / c + 2.0 + 0.05 * c);
    if (best == 0 || cost < best_cost) {
      best = c;
      best_n = n;
      best_cost = cost;
    }
  }
  *clusters_out = best_n;
  return best;
}

static int encode_decode_maps(const Dims& dm, const void* q, const void* K, const void* V, unsigned q_rows,
                              CUtensorMap* tmK, CUtensorMap* tmV, CUtensorMap* tmQ, TensorMapEncodeFn encode) {
  const cuuint64_t gdim[2] = {(cuuint64_t)dm.D, (cuuint64_t)dm.units * (cuuint64_t)dm.cap};
  const cuuint64_t gstride[1] = {(cuuint64_t)dm.D * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)decode::kT};
  const cuuint32_t estride[2] = {1, 1};
  for (int i = 0; i < 3; ++i) {
    // K, V: boxes of 64 channels x 128 tokens; q: 64 channels x q_rows rows (a unit's heads, padded by its
    // neighbours' or by zeros)
    const cuuint64_t qdim[2] = {(cuuint64_t)dm.D, (cuuint64_t)dm.B * (cuuint64_t)dm.Hq};
    const cuuint32_t qbox[2] = {64, q_rows};
    CUresult r = encode(i == 0 ? tmK : (i == 1 ? tmV : tmQ), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                        const_cast<void*>(i == 0 ? K : (i == 1 ? V : q)), i < 2 ? gdim : qdim, gstride, i < 2 ? box : qbox,
                        estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
      snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
      return CAOTE_ERR_CUDA;
    }
  }
  return CAOTE_OK;
}

static int launch_decode_cluster(const Dims& dm, const void* q, const void* K, const void* V, const int* len,
                                 float* base, float* o, float* scores, char* ws, cudaStream_t st, bool* used,
                                 const float* vsum = nullptr) {
  *used = false;
  TensorMapEncodeFn encode = tensor_map_encoder();
  const bool carried = dm.base_mode == CAOTE_BASE_ACCUM || dm.base_mode == CAOTE_BASE_EXTERNAL;
  if (!encode || (carried && !aligned(base, 16)) || !aligned(q, 16)) return CAOTE_OK;
  const ClusterKernel kernel = cluster_kernel(dm.G, dm.base_mode);
  // (the attributes below are per function: every instantiation gets them the first time it is used)
  static std::mutex attr_mu;
  static std::vector<std::pair<int, ClusterKernel>> attr_done;
  {
    int dev = 0;
    CAOTE_CUDA(cudaGetDevice(&dev));
    std::lock_guard<std::mutex> lk(attr_mu);
    bool done = false;
    for (auto& e : attr_done) done |= (e.first == dev && e.second == kernel);
    if (!done) {
      CAOTE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dcl::smem_bytes()));
      CAOTE_CUDA(cudaFuncSetAttribute(kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
      attr_done.push_back({dev, kernel});
    }
  }
  int clusters = 0;
  const int c = choose_cluster(dm, kernel, &clusters);
  if (c == 0) return CAOTE_OK;
  CUtensorMap tmK, tmV, tmQ;
  int rc = encode_decode_maps(dm, q, K, V, 8, &tmK, &tmV, &tmQ, encode);
  if (rc) return rc;
  if (clusters > dm.units) clusters = dm.units;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(clusters * c));
  cfg.blockDim = dim3(dcl::kThreads);
  cfg.dynamicSmemBytes = dcl::smem_bytes();
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)c;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // (the kernel starts with ptx::pdl_wait)
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 2;
  int* status = reinterpret_cast<int*>(ws);
  const long long wait_cycles = g_wait_cycles.load(std::memory_order_relaxed);
  CAOTE_LAUNCH("decode_cluster_kernel", st, {
    cudaError_t e = cudaLaunchKernelEx(&cfg, kernel, tmK, tmV, tmQ, dm, len, base, o, scores, status,
                                       wait_cycles, vsum);
    if (e != cudaSuccess) return cuda_fail(e, "decode_cluster_kernel");
  });
  *used = true;
  return CAOTE_OK;
}

static int launch_decode_score(const Dims& dm, const void* q, const void* K, const void* V, const int* len,
                               float* base, float* o, float* scores, int* status, char* scratch, float* rowstat,
                               int stat_tag, int grid_cap, cudaStream_t st, bool* used, const float* vsum) {
  // status: the workspace header; scratch: where the plan and the records go; rowstat: [units][kHeadStatFloats], first 8 of a unit for the heads'
  // log-sum-exp (or null); stat_tag: what the header's statistics tag becomes (< 0: left alone);
  // grid_cap > 0: at most that many CTAs (when the kernel shares the GPU with the cluster kernel)
  *used = false;
  int grid_limit = decode_grid_limit();
  if (grid_cap > 0 && grid_limit > grid_cap) grid_limit = grid_cap;
  TensorMapEncodeFn encode = tensor_map_encoder();
  const bool carried = dm.base_mode == CAOTE_BASE_ACCUM || dm.base_mode == CAOTE_BASE_EXTERNAL;
  if (grid_limit <= 0 || !encode || (carried && !aligned(base, 16)) || !aligned(q, 16)) return CAOTE_OK;
  decode::Plan pl;
  decode::carve(dm, scratch, &pl, grid_limit);
  pl.rowstat = rowstat;
  pl.stat_tag = stat_tag;
  CUtensorMap tmK, tmV, tmQ;
  const cuuint64_t gdim[2] = {(cuuint64_t)dm.D, (cuuint64_t)dm.units * (cuuint64_t)dm.cap};
  const cuuint64_t gstride[1] = {(cuuint64_t)dm.D * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)decode::kT};
  const cuuint32_t estride[2] = {1, 1};
  for (int i = 0; i < 2; ++i) {
    CUresult r = encode(i == 0 ? &tmK : &tmV, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(i == 0 ? K : V), gdim,
                        gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
      snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
      return CAOTE_ERR_CUDA;
    }
  }
  {
    // the query rows: boxes of 64 channels x 16 rows (a unit's heads, padded by its neighbours' or by zeros)
    const cuuint64_t qdim[2] = {(cuuint64_t)dm.D, (cuuint64_t)dm.B * (cuuint64_t)dm.Hq};
    const cuuint32_t qbox[2] = {64, 16};
    CUresult r = encode(&tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(q), qdim, gstride, qbox, estride,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
      snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
      return CAOTE_ERR_CUDA;
    }
  }
  CAOTE_LAUNCH("decode_plan_kernel", st,
               launch_pdl(decode::plan_kernel, dim3(1), dim3(1024), 0, st, dm.units, dm.Hkv, dm.cap, len, pl, status));
  const int tiles_per_unit = (dm.cap + decode::kT - 1) / decode::kT;
  const long long max_items = (long long)dm.units * ((tiles_per_unit + pl.tpi - 1) / pl.tpi);
  const int grid = (int)(max_items < grid_limit ? max_items : grid_limit);
  if (!vsum) {
    CAOTE_LAUNCH("decode_tc_kernel", st,
                 launch_pdl(decode::decode_tc_kernel<false>, dim3(grid), dim3(decode::kTcThreads), decode::tc_smem_bytes(false), st, 
                     tmK, tmV, tmQ, dm, len, base, o, scores, nullptr, pl, status));
  } else {
    // FastCAOTE: one pass over K and V, then scores from the stored logits and distances
    CAOTE_LAUNCH("decode_tc_fast_kernel", st,
                 launch_pdl(decode::decode_tc_kernel<true>, dim3(grid), dim3(decode::kTcThreads), decode::tc_smem_bytes(true), st, 
                     tmK, tmV, tmQ, dm, len, base, o, scores, vsum, pl, status));
    dim3 fgrid(tiles_per_unit, dm.units);
    CAOTE_LAUNCH("fast_finish_kernel", st, launch_pdl(decode::fast_finish_kernel, dim3(fgrid), dim3(decode::kT), 0, st, dm, len, base, scores, pl));
  }
  *used = true;
  return CAOTE_OK;
}


// The heads' statistics of every unit ([units][kHeadStatFloats] floats) sit right behind the workspace header on the single-
// query paths; the streaming kernel's plan and records follow it.
static size_t rowstat_bytes(const Dims& dm) { return align_up(sizeof(float) * kHeadStatFloats * (size_t)dm.units, 256); }

// The same problem restricted to `count` sequences (the caller offsets the pointers).
static Dims sub_dims(const Dims& dm, int count) {
  Dims d = dm;
  d.B = count;
  d.units = count * dm.Hkv;
  return d;
}

// SMs the cluster kernel occupies on these dimensions.
static int side_clusters_sms(const Dims& d, int base_mode) {
  int n = 0;
  const int c = choose_cluster(d, cluster_kernel(d.G, base_mode), &n);
  if (n > d.units) n = d.units;
  return c * n;
}

// ---- two kernels side by side --------------------------------------------------------------------------------
// A cluster of C CTAs takes one unit at a time, the GPU holds n such clusters, and n C is often well below the SM
// count (a cluster lives inside one GPC) while units / n is rarely whole: the last round runs a few clusters and
// the SMs outside the clusters idle throughout. When that costs enough, the last `tail` sequences of the batch go
// to the streaming kernel instead, on a second stream and on as many CTAs as there are SMs outside the clusters, at
// the same time as the cluster kernel works on the others. Returns the number of tail sequences (0: one kernel).
// The estimates only rank the options; rates in bytes per second per SM and per cluster round are measured ones.
static int plan_side_by_side(const Dims& dm, int base_mode) {
  const int mode = g_side_by_side.load(std::memory_order_relaxed);
  if (mode == 0 || dm.B < 2) return 0;
  if (mode >= 2) {  // forced: the last mode - 1 sequences, if the cluster kernel can take the others
    const int tail = mode - 1 < dm.B ? mode - 1 : dm.B - 1;
    return side_clusters_sms(sub_dims(dm, dm.B - tail), base_mode) > 0 ? tail : 0;
  }
  const double unit_bytes = (double)dm.cap * dm.D * 4.0;  // K and V rows, bf16
  // measured: the cluster kernel moves about 33 GB/s of K and V per SM it occupies (3.7 TB/s on 112 SMs, 4.5 on 135);
  // the streaming kernel beside it about 15 GB/s per SM (8 units of 16 385 tokens on 36 SMs in 118 us), after some
  // 15 us for its plan launch and pipeline fill
  const double cluster_rate_per_sm = 33e9, stream_rate_per_sm = 15e9, stream_fixed = 15e-6;
  auto cluster_time = [&](int seqs, int* idle) {
    const Dims d = sub_dims(dm, seqs);
    int n = 0;
    const int c = choose_cluster(d, cluster_kernel(dm.G, base_mode), &n);
    if (c == 0 || n == 0) return -1.0;
    if (n > d.units) n = d.units;
    *idle = g_sm_count - n * c;
    const long long rounds = ((long long)d.units + n - 1) / n;
    return (double)rounds * (unit_bytes * n / (cluster_rate_per_sm * n * c));
  };
  int idle = 0;
  const double alone = cluster_time(dm.B, &idle);
  if (alone <= 0.0) return 0;
  int best = 0;
  // Worth it only for an estimated 10 % or more: the join delays whatever follows, and the cluster kernel itself
  // slows down a little next to a second kernel (256 ragged units of about 7 k tokens with 13 SMs outside the
  // clusters: 204 us with 16 units moved away against 209 us with all of them, no gain left after the join).
  double best_t = alone * 0.90;
  for (int tail = 1; tail < dm.B && tail <= 16; ++tail) {
    const double tc = cluster_time(dm.B - tail, &idle);
    if (tc <= 0.0 || idle < 8) continue;
    const double ts = stream_fixed + (double)tail * dm.Hkv * unit_bytes / (idle * stream_rate_per_sm);
    const double t = tc > ts ? tc : ts;
    if (t < best_t) {
      best_t = t;
      best = tail;
    }
  }
  return best;
}

// The second stream and the two events of the fork and the join, one set per device, made on first use.
struct SideStream {
  cudaStream_t stream = nullptr;
  cudaEvent_t fork = nullptr, join = nullptr;
};
static std::mutex g_side_mu;
static int side_stream(SideStream* out) {
  static SideStream per_dev[64];
  int dev = 0;
  CAOTE_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return CAOTE_ERR_UNSUPPORTED;
  SideStream& ss = per_dev[dev];
  if (!ss.stream) {
    CAOTE_CUDA(cudaStreamCreateWithFlags(&ss.stream, cudaStreamNonBlocking));
    CAOTE_CUDA(cudaEventCreateWithFlags(&ss.fork, cudaEventDisableTiming));
    CAOTE_CUDA(cudaEventCreateWithFlags(&ss.join, cudaEventDisableTiming));
  }
  *out = ss;
  return CAOTE_OK;
}

// The sum-of-errors pass that follows the cluster kernel on single-query shapes.
template <int G>
static int launch_sum_errors_decode_g(const Dims& dm, const CUtensorMap& tmK, const CUtensorMap& tmV, const void* q,
                                      const int* len, const float* o, float* scores, char* ws, cudaStream_t st) {
  int rc = allow_smem(sed::sum_errors_decode_kernel<G>, sed::smem_bytes());
  if (rc) return rc;
  dim3 grid((dm.cap + sed::kT - 1) / sed::kT, dm.units);
  CAOTE_LAUNCH("sum_errors_decode_kernel", st,
               launch_pdl(sed::sum_errors_decode_kernel<G>, grid, dim3(sed::kThreads), sed::smem_bytes(), st, tmK, tmV, dm,
                          (const __nv_bfloat16*)q, len, o, reinterpret_cast<const float*>(ws + kHeaderBytes), scores,
                          reinterpret_cast<int*>(ws)));
  return CAOTE_OK;
}
static int launch_sum_errors_decode(const Dims& dm, const void* q, const void* K, const void* V, const int* len,
                                    const float* o, float* scores, char* ws, cudaStream_t st) {
  TensorMapEncodeFn encode = tensor_map_encoder();
  if (!encode) return CAOTE_ERR_CUDA;  // (the cluster kernel before it was launched with the same encoder)
  CUtensorMap tmK, tmV, tmQ;
  int rc = encode_decode_maps(dm, q, K, V, 8, &tmK, &tmV, &tmQ, encode);
  if (rc) return rc;
  switch (dm.G) {
    case 1: return launch_sum_errors_decode_g<1>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 2: return launch_sum_errors_decode_g<2>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 3: return launch_sum_errors_decode_g<3>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 4: return launch_sum_errors_decode_g<4>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 5: return launch_sum_errors_decode_g<5>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 6: return launch_sum_errors_decode_g<6>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 7: return launch_sum_errors_decode_g<7>(dm, tmK, tmV, q, len, o, scores, ws, st);
    case 8: return launch_sum_errors_decode_g<8>(dm, tmK, tmV, q, len, o, scores, ws, st);
    default: return CAOTE_ERR_UNSUPPORTED;
  }
}

// Shapes the tensor-core prefill kernels cover.
static bool prefill_shape_ok(const caote_params_t* p) {
  const int G = p->n_q_heads / p->n_kv_heads;
  return p->dtype == CAOTE_BF16 && p->head_dim == 128 && p->base_mode == CAOTE_BASE_CHUNK_SUM && p->n_new >= 16 && p->scale > 0.f &&
         (long long)G * p->n_new >= 64 && (long long)p->batch * p->n_kv_heads * p->capacity < (1LL << 31) &&
         (long long)p->batch * p->n_q_heads * p->n_new < (1LL << 31);
}

static int encode_rows_map(CUtensorMap* tm, const void* ptr, unsigned long long rows, TensorMapEncodeFn encode,
                           unsigned box_rows = 128) {
  const cuuint64_t gdim[2] = {128, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {256};
  const cuuint32_t box[2] = {64, box_rows};
  const cuuint32_t estride[2] = {1, 1};
  CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim, gstride, box, estride,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(g_cuda_error, sizeof(g_cuda_error), "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
    return CAOTE_ERR_CUDA;
  }
  return CAOTE_OK;
}

static int launch_prefill_score(const Dims& dm, const void* q, const void* K, const void* V, const int* len, float* o,
                                float* scores, char* ws, cudaStream_t st, bool* used, const float* vsum) {
  *used = false;
  TensorMapEncodeFn encode = tensor_map_encoder();
  if (!encode) return CAOTE_OK;
  prefill::Scratch sc;
  prefill::carve(dm, ws + kHeaderBytes, &sc);
  int* status = reinterpret_cast<int*>(ws);
  CUtensorMap tmQ, tmK, tmK64, tmV64;
  int rc = encode_rows_map(&tmQ, q, (unsigned long long)dm.B * dm.Hq * dm.m, encode);
  if (!rc) rc = encode_rows_map(&tmK, K, (unsigned long long)dm.units * dm.cap, encode);
  if (!rc) rc = encode_rows_map(&tmK64, K, (unsigned long long)dm.units * dm.cap, encode, prefill::kKeys);
  if (!rc) rc = encode_rows_map(&tmV64, V, (unsigned long long)dm.units * dm.cap, encode, prefill::kKeys);
  if (rc) return rc;
  rc = allow_smem(prefill::attn_kernel, prefill::attn_smem_bytes());
  if (!rc) rc = allow_smem(prefill::score_kernel, prefill::score_smem_bytes());
  if (rc) return rc;
  {
    dim3 grid((dm.R + prefill::kTile - 1) / prefill::kTile, dm.units, sc.nsplit);
    CAOTE_LAUNCH("prefill_attn_kernel", st,
                 launch_pdl(prefill::attn_kernel, dim3(grid), dim3(prefill::kAttnThreads), prefill::attn_smem_bytes(), st, tmQ, tmK64, tmV64, dm, len,
                                                                                                    sc, o, status));
  }
  const bool merged_with_mean = !vsum;  // the splits' merge (if there are splits) and the column mean in one launch
  if (merged_with_mean) {
    dim3 grid(dm.units, prefill::kD / 16);
    CAOTE_LAUNCH("prefill_combine_xsum_kernel", st,
                 launch_pdl(prefill::attn_combine_xsum_kernel, dim3(grid), dim3(prefill::kCxThreads), 0, st, dm, len, sc, o));
  } else if (sc.nsplit > 1) {
    dim3 grid((dm.R + 3) / 4, dm.units);
    CAOTE_LAUNCH("prefill_attn_combine_kernel", st, launch_pdl(prefill::attn_combine_kernel, dim3(grid), dim3(4 * prefill::kD), 0, st, dm, len, sc, o));
  }
  if (vsum) {
    CAOTE_LAUNCH("fast_mean_kernel", st, fast::mean_kernel<<<dm.units, prefill::kD, 0, st>>>(dm.Hkv, dm.cap, prefill::kD, len, vsum, sc.X));
  }
  {
    dim3 grid((dm.cap + prefill::kScoreKeys - 1) / prefill::kScoreKeys, dm.units);
    CAOTE_LAUNCH("prefill_score_kernel", st,
                 launch_pdl(prefill::score_kernel, dim3(grid), dim3(prefill::kScoreThreads), prefill::score_smem_bytes(), st, 
                     tmQ, tmK, tmV64, dm, len, sc, scores, status));
  }
  *used = true;
  return CAOTE_OK;
}

// The split heuristics of the prefill and any-shape paths look at the SM count: keep it current for this device
// (cached per device; left at its default when there is no device, e.g. when only sizes are asked for).
static void refresh_sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    (void)cudaGetLastError();
    return;
  }
  int n = cached[dev].load(std::memory_order_acquire);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      return;
    }
    cached[dev].store(n, std::memory_order_release);
  }
  g_sm_count = n;
}

static size_t workspace_bytes(const caote_params_t* p) {
  refresh_sm_count();
  const Dims dm = make_dims(p);
  size_t need = generic::carve(dm, nullptr, nullptr);
  if (decode_shape_ok(p)) {
    const size_t need2 = rowstat_bytes(dm) + decode::carve(dm, nullptr, nullptr, 0);
    if (need2 > need) need = need2;
  }
  if (prefill_shape_ok(p)) {
    const size_t need3 = prefill::carve(dm, nullptr, nullptr);
    if (need3 > need) need = need3;
  }
  return kHeaderBytes + need;
}

// ---- built-in scratch of caote_score_static ------------------------------------------------------
// Lives in the library's device image: every GPU that loads the library holds these bytes until the
// process exits. The name below is only a host-side handle; the device address is looked up once per
// device with cudaGetSymbolAddress.
constexpr size_t kStaticScratchBytes = CAOTE_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static int static_scratch_address(char** out) {
  static std::mutex mu;
  static char* addr[64] = {};
  int dev = 0;
  CAOTE_CUDA(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return CAOTE_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lk(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    CAOTE_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
    if (!p) return CAOTE_ERR_CUDA;
    addr[dev] = static_cast<char*>(p);
  }
  *out = addr[dev];
  return CAOTE_OK;
}

template <typename T, int D>
static int launch_post_evict(const Dims& dm, const void* q, const void* K, const void* V, const int* len,
                             const int* evict_idx, int max_evict, const int* n_evict, const float* o, float* o_post,
                             const char* ws, cudaStream_t st) {
  const size_t smem = post::smem_bytes<D>();
  int rc = allow_smem(post::post_evict_kernel<T, D>, smem);
  if (rc) return rc;
  const int* tag = ws ? reinterpret_cast<const int*>(ws) + kStatTagIndex : nullptr;
  const float* stats = ws ? reinterpret_cast<const float*>(ws + kHeaderBytes) : nullptr;
  const int stat_stride = (dm.R + prefill::kTile - 1) / prefill::kTile * prefill::kTile;
  // Blocks of queries in bf16 / d 128 may have per-row statistics in the workspace (only the device knows which path
  // scored them): the kernel for that case goes first and returns at once if they are not there; the general
  // kernel after it returns at once if they are.
  int rows_kernel = 0;
  if constexpr (std::is_same<T, __nv_bfloat16>::value && D == 128) {
    if (ws && dm.m > 1 && aligned(o, 16) && aligned(o_post, 16)) {
      rc = allow_smem(post::post_evict_rows_kernel, post::rows_smem_bytes());
      if (rc) return rc;
      dim3 rgrid((dm.R + post::kBlockRows - 1) / post::kBlockRows, dm.units);
      CAOTE_LAUNCH("post_evict_rows_kernel", st, post::post_evict_rows_kernel<<<rgrid, 256, post::rows_smem_bytes(), st>>>(
          dm, (const T*)q, (const T*)K, (const T*)V, len, evict_idx, max_evict, n_evict, o, o_post, tag, stats, stat_stride));
      rows_kernel = 1;
    }
  }
  dim3 grid((dm.R + post::kRows - 1) / post::kRows, dm.units);
  CAOTE_LAUNCH("post_evict_kernel", st, post::post_evict_kernel<T, D><<<grid, 32 * post::kRows, smem, st>>>(
      dm, (const T*)q, (const T*)K, (const T*)V, len, evict_idx, max_evict, n_evict, o, o_post, tag, stats, stat_stride,
      rows_kernel));
  return CAOTE_OK;
}

template <typename T, int D>
static int launch_greedy(const Dims& dm, const void* V, const float* h, const int* len, const int* budget, const int* pos,
                         int* evict_idx, int* order, int max_evict, int* n_evict, int* status, cudaStream_t st) {
  const size_t smem = greedy::smem_bytes(dm.cap, D);
  int rc = allow_smem(greedy::greedy_kernel<T, D>, smem);
  if (rc) return rc;
  CAOTE_LAUNCH("greedy_select_kernel", st, greedy::greedy_kernel<T, D><<<dm.units, greedy::kThreads, smem, st>>>(
      dm.Hkv, dm.cap, (const T*)V, h, len, budget, pos, evict_idx, order, max_evict, n_evict, status));
  return CAOTE_OK;
}

// Greedy eviction with the unit's value rows in the shared memory of a cluster (bf16, d 128; what 16 CTAs cannot
// hold of a long unit stays in global memory and is swept from L2). *used = false: the shape does not fit (more
// than 16 x 2048 tokens, or no cluster can run) or the one-CTA kernel is the better choice, and the caller takes that. Among the cluster sizes that hold a unit, the largest one of which the GPU can run as
// many at once as there are units: more CTAs per unit make a pick faster, a second wave of clusters makes the call
// twice as long.
static int launch_greedy_cluster(const Dims& dm, const void* V, const float* h, const int* len, const int* budget,
                                 const int* pos, int* evict_idx, int* order, int max_evict, int* n_evict, int* status,
                                 cudaStream_t st, bool* used) {
  *used = false;
  if (!aligned(V, 16)) return CAOTE_OK;
  int need = 1;  // the smallest cluster that holds the unit in shared memory, else the largest cluster
  while (need < greedy_cl::kMaxC && (dm.cap + need - 1) / need > greedy_cl::kMaxRows) need *= 2;
  if ((dm.cap + need - 1) / need > greedy_cl::kMaxShare) return CAOTE_OK;
  // (the function's limits are set to the largest any launch may ask for, the same value every time: calls from
  // several host threads then never see a limit below what they need)
  CAOTE_CUDA(cudaFuncSetAttribute(greedy_cl::greedy_cluster_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
  CAOTE_CUDA(cudaFuncSetAttribute(greedy_cl::greedy_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)greedy_cl::smem_bytes(greedy_cl::kMaxRows, greedy_cl::kMaxShare)));
  int best_c = 0, best_rows = 0, best_got = 0;
  for (int c = need; c <= greedy_cl::kMaxC; c *= 2) {
    const int rows = ((dm.cap + c - 1) / c + 7) / 8 * 8;
    const size_t smem = greedy_cl::smem_bytes(rows < greedy_cl::kMaxRows ? rows : greedy_cl::kMaxRows, rows);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(c * dm.units));
    cfg.blockDim = dim3(greedy_cl::kThreads);
    cfg.dynamicSmemBytes = smem;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = (unsigned)c;
    at[0].val.clusterDim.y = 1;
    at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    int got = 0;
    if (cudaOccupancyMaxActiveClusters(&got, greedy_cl::greedy_cluster_kernel, &cfg) != cudaSuccess || got <= 0) {
      (void)cudaGetLastError();
      continue;
    }
    if (best_c == 0 || got >= dm.units) {
      best_c = c;
      best_rows = rows;
      best_got = got;
    }
    if (got < dm.units && best_c != c) break;  // larger clusters only fit fewer at once
  }
  if (best_c == 0) return CAOTE_OK;
  {
    // Worth it? Per pick the one-CTA kernel sweeps the unit's rows from L2 (measured: 19 us at 4224 rows, taken as
    // 3 us + 3.8 ns per row), this one its share of them from shared memory plus a cluster barrier (measured: 5.25 us at
    // 528 rows per CTA, 8.35 us at 768 + 288 left in global memory: about 4.2 us + 2 ns per row + 9 ns per row from
    // L2); but the GPU runs fewer clusters at once than single CTAs, and with a handful of picks loading the rows is
    // all there is.
    const int in_smem = best_rows < greedy_cl::kMaxRows ? best_rows : greedy_cl::kMaxRows;
    const double t_one = 3.0 + 0.0038 * dm.cap, t_cluster = 4.2 + 0.002 * in_smem + 0.009 * (best_rows - in_smem);
    const double waves_one = (double)((dm.units + g_sm_count - 1) / g_sm_count);
    const double waves_cluster = (double)((dm.units + best_got - 1) / best_got);
    if (max_evict < 4 || t_one * waves_one < 1.2 * t_cluster * waves_cluster) return CAOTE_OK;
  }
  const int rows_smem = best_rows < greedy_cl::kMaxRows ? best_rows : greedy_cl::kMaxRows;
  const size_t smem = greedy_cl::smem_bytes(rows_smem, best_rows);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(best_c * dm.units));
  cfg.blockDim = dim3(greedy_cl::kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)best_c;
  at[0].val.clusterDim.y = 1;
  at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  CAOTE_LAUNCH("greedy_cluster_kernel", st, {
    cudaError_t e = cudaLaunchKernelEx(&cfg, greedy_cl::greedy_cluster_kernel, dm.Hkv, dm.cap, best_rows, rows_smem,
                                       (const __nv_bfloat16*)V, h, len, budget, pos, evict_idx, order, max_evict, n_evict,
                                       status);
    if (e != cudaSuccess) return cuda_fail(e, "greedy_cluster_kernel");
  });
  *used = true;
  return CAOTE_OK;
}

}  // namespace caote

using namespace caote;

extern "C" {

// Host-side checks of caote_append / caote_score arguments; nothing is enqueued before they pass.
static int append_args_check(const caote_params_t* p, const void* K, const void* V, const int32_t* len, const void* k_new,
                             const void* v_new, const void* workspace, size_t workspace_bytes_) {
  if (!params_ok(p) || !K || !V || !len || !k_new || !v_new || !workspace) return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  if (workspace_bytes_ < kHeaderBytes || !aligned(workspace, 256)) return CAOTE_ERR_INVALID_ARG;
  if (!aligned(K, 16) || !aligned(V, 16) || !aligned(k_new, 16) || !aligned(v_new, 16)) return CAOTE_ERR_INVALID_ARG;
  return CAOTE_OK;
}
static int score_args_check(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                            const float* base, const float* o, const float* scores) {
  if (!params_ok(p) || !q || !K || !V || !len || !o || !scores) return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  if ((p->base_mode == CAOTE_BASE_ACCUM || p->base_mode == CAOTE_BASE_EXTERNAL) && !base)
    return CAOTE_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(o, 16)) return CAOTE_ERR_INVALID_ARG;
  return CAOTE_OK;
}
static int score_workspace_check(const caote_params_t* p, const void* workspace, size_t workspace_bytes_) {
  if (!workspace || workspace_bytes_ < workspace_bytes(p) || !aligned(workspace, 256)) return CAOTE_ERR_INVALID_ARG;
  return CAOTE_OK;
}

size_t caote_workspace_bytes(const caote_params_t* params) {
  if (!params_ok(params) || !params_supported(params)) return 0;
  return workspace_bytes(params);
}

// Whether the append of this shape runs a CTA per sequence, and can then also add the one new value row of every unit
// to FastCAOTE's running sum (m = 1).
static bool append_per_sequence(const Dims& dm) { return dm.Hkv * dm.m <= 16; }

// caote_append, and the append inside caote_step_fast (vsum: the units' running sums, folded in where
// append_per_sequence(dm) and m = 1).
static int append_impl(const caote_params_t* p, void* K, void* V, float* base, int32_t* pos, int32_t* len,
                       int32_t* n_seen, const void* k_new, const void* v_new, void* workspace,
                       size_t workspace_bytes_, caote_stream_t stream, float* vsum) {
  int rc = append_args_check(p, K, V, len, k_new, v_new, workspace, workspace_bytes_);
  if (rc) return rc;
  rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  const int row_bytes = dm.D * (p->dtype == CAOTE_BF16 ? 2 : 4);
  cudaStream_t st = (cudaStream_t)stream;
  if (append_per_sequence(dm)) {  // (single-query decode: a CTA per sequence, which moves its lengths on itself)
    CAOTE_LAUNCH("append_seq_kernel", st,
                 launch_pdl(sel::append_seq_kernel, dim3(dm.B), dim3(64 * dm.Hkv * dm.m), 0, st, dm.Hkv, dm.cap, dm.m,
                            row_bytes, (char*)K, (char*)V, base, pos, len, n_seen, (const char*)k_new,
                            (const char*)v_new, (int*)workspace, dm.m == 1 ? vsum : nullptr,
                            p->dtype == CAOTE_BF16 ? 2 : 4));
    return CAOTE_OK;
  }
  CAOTE_LAUNCH("append_kernel", st, launch_pdl(sel::append_kernel, dim3(dim3(dm.units, (dm.m + 7) / 8)), dim3(256), 0, st, dm.Hkv, dm.cap, dm.m, row_bytes, (char*)K, (char*)V, base, pos,
                                               len, n_seen, (const char*)k_new, (const char*)v_new,
                                               (int*)workspace, dm.B, (int*)workspace + 4));
  return CAOTE_OK;
}

int caote_append(const caote_params_t* p, void* K, void* V, float* base, int32_t* pos, int32_t* len,
                 int32_t* n_seen, const void* k_new, const void* v_new, void* workspace,
                 size_t workspace_bytes_, caote_stream_t stream) {
  return append_impl(p, K, V, base, pos, len, n_seen, k_new, v_new, workspace, workspace_bytes_, stream, nullptr);
}

// caote_score (vsum == NULL) and caote_score_fast (vsum: the per-unit sums of the cached value rows).
static int score_impl(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                      float* base, const float* vsum, float* o, float* scores, void* workspace, size_t workspace_bytes_,
                      caote_stream_t stream, bool allow_side_stream = true) {
  int rc = score_args_check(p, q, K, V, len, base, o, scores);
  if (!rc) rc = score_workspace_check(p, workspace, workspace_bytes_);
  if (!rc) rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  if (decode_shape_ok(p)) {
    bool used = false;
    int* status = reinterpret_cast<int*>(ws);
    float* rowstat = reinterpret_cast<float*>(ws + kHeaderBytes);
    char* scratch = ws + kHeaderBytes + rowstat_bytes(dm);
    if (!vsum) {
      const bool carried = dm.base_mode == CAOTE_BASE_ACCUM || dm.base_mode == CAOTE_BASE_EXTERNAL;
      const int tail = (allow_side_stream && decode_grid_limit() > 0 && tensor_map_encoder() && aligned(q, 16) &&
                        (!carried || aligned(base, 16))) ? plan_side_by_side(dm, dm.base_mode) : 0;
      if (tail > 0) {
        // the first B - tail sequences on the cluster kernel, the last `tail` on the streaming kernel beside it
        const int head = dm.B - tail;
        const Dims dh = sub_dims(dm, head), dt = sub_dims(dm, tail);
        SideStream ss;
        std::lock_guard<std::mutex> lk(g_side_mu);
        TraceScope region("decode_side_by_side", st);  // (tracing: the time from the fork to the join)
        rc = side_stream(&ss);
        if (rc) return rc;
        CAOTE_CUDA(cudaEventRecord(ss.fork, st));
        CAOTE_CUDA(cudaStreamWaitEvent(ss.stream, ss.fork, 0));
        rc = launch_decode_cluster(dh, q, K, V, len, base, o, scores, ws, st, &used);
        if (rc) return rc;
        if (used) {
          const size_t uo = (size_t)head * dm.Hkv, qo = (size_t)head * dm.Hq * dm.D;
          bool used_t = false;
          rc = launch_decode_score(dt, (const __nv_bfloat16*)q + qo, (const __nv_bfloat16*)K + uo * dm.cap * dm.D,
                                   (const __nv_bfloat16*)V + uo * dm.cap * dm.D, len + head, base ? base + uo * dm.cap : nullptr,
                                   o + qo, scores + uo * dm.cap, status, scratch, rowstat + uo * kHeadStatFloats, -1,
                                   g_sm_count - side_clusters_sms(dh, dm.base_mode), ss.stream, &used_t, nullptr);
          if (!rc && !used_t) rc = CAOTE_ERR_CUDA;  // (its preconditions were checked above)
          const cudaError_t e1 = cudaEventRecord(ss.join, ss.stream);
          const cudaError_t e2 = cudaStreamWaitEvent(st, ss.join, 0);
          if (rc) return rc;
          if (e1 != cudaSuccess) return cuda_fail(e1, "cudaEventRecord");
          if (e2 != cudaSuccess) return cuda_fail(e2, "cudaStreamWaitEvent");
          return CAOTE_OK;
        }
      }
      rc = launch_decode_cluster(dm, q, K, V, len, base, o, scores, ws, st, &used);
      if (rc || used) return rc;
    } else {
      // FastCAOTE: the same kernel with the mean of the value rows in the place of X
      rc = launch_decode_cluster(dm, q, K, V, len, base, o, scores, ws, st, &used, vsum);
      if (rc || used) return rc;
    }
    rc = launch_decode_score(dm, q, K, V, len, base, o, scores, status, scratch, rowstat, kStatPerHead, 0, st, &used, vsum);
    if (rc || used) return rc;
  }
  if (prefill_shape_ok(p)) {
    bool used = false;
    rc = launch_prefill_score(dm, q, K, V, len, o, scores, ws, st, &used, vsum);
    if (rc || used) return rc;
  }
  if (p->dtype == CAOTE_BF16) {
    if (dm.D == 128) return launch_generic_score<__nv_bfloat16, 128>(dm, q, K, V, len, base, o, scores, ws, st, vsum);
    return launch_generic_score<__nv_bfloat16, 64>(dm, q, K, V, len, base, o, scores, ws, st, vsum);
  }
  if (dm.D == 128) return launch_generic_score<float, 128>(dm, q, K, V, len, base, o, scores, ws, st, vsum);
  return launch_generic_score<float, 64>(dm, q, K, V, len, base, o, scores, ws, st, vsum);
}

int caote_score(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                float* base, float* o, float* scores, void* workspace, size_t workspace_bytes_,
                caote_stream_t stream) {
  return score_impl(p, q, K, V, len, base, nullptr, o, scores, workspace, workspace_bytes_, stream);
}

int caote_score_sum_errors(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                           float* o, float* scores, void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  if (!params_ok(p) || !q || !K || !V || !len || !o || !scores || !workspace) return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  if (p->base_mode != CAOTE_BASE_LAST_QUERY && p->base_mode != CAOTE_BASE_CHUNK_SUM) return CAOTE_ERR_UNSUPPORTED;
  if (workspace_bytes_ < workspace_bytes(p) || !aligned(workspace, 256)) return CAOTE_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(K, 16) || !aligned(V, 16) || !aligned(o, 16)) return CAOTE_ERR_INVALID_ARG;
  int rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  if (decode_shape_ok(p)) {
    // one query per head: the cluster kernel for o and the heads' statistics, then one more pass over K and V
    bool used = false;
    rc = launch_decode_cluster(dm, q, K, V, len, nullptr, o, scores, ws, st, &used);
    if (rc) return rc;
    if (used) return launch_sum_errors_decode(dm, q, K, V, len, o, scores, ws, st);
  }
  if (p->dtype == CAOTE_BF16) {
    if (dm.D == 128) return launch_generic_score<__nv_bfloat16, 128>(dm, q, K, V, len, nullptr, o, scores, ws, st, nullptr, true);
    return launch_generic_score<__nv_bfloat16, 64>(dm, q, K, V, len, nullptr, o, scores, ws, st, nullptr, true);
  }
  if (dm.D == 128) return launch_generic_score<float, 128>(dm, q, K, V, len, nullptr, o, scores, ws, st, nullptr, true);
  return launch_generic_score<float, 64>(dm, q, K, V, len, nullptr, o, scores, ws, st, nullptr, true);
}

int caote_score_fast(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                     float* base, const float* vsum, float* o, float* scores, void* workspace,
                     size_t workspace_bytes_, caote_stream_t stream) {
  if (!vsum || !aligned(vsum, 16)) return CAOTE_ERR_INVALID_ARG;
  return score_impl(p, q, K, V, len, base, vsum, o, scores, workspace, workspace_bytes_, stream);
}

int caote_vsum(const caote_params_t* p, const void* V, const int32_t* len, float* vsum, caote_stream_t stream) {
  if (!params_ok(p) || !V || !len || !vsum) return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  int rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  cudaStream_t st = (cudaStream_t)stream;
  if (p->dtype == CAOTE_BF16) {
    CAOTE_LAUNCH("fast_vsum_kernel", st, fast::vsum_kernel<__nv_bfloat16><<<dm.units, 256, 0, st>>>(
        dm.Hkv, dm.cap, dm.D, (const __nv_bfloat16*)V, len, vsum));
  } else {
    CAOTE_LAUNCH("fast_vsum_kernel", st, fast::vsum_kernel<float><<<dm.units, 256, 0, st>>>(dm.Hkv, dm.cap, dm.D, (const float*)V, len, vsum));
  }
  return CAOTE_OK;
}

int caote_score_static(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                       float* base, float* o, float* scores, int32_t* status_out, caote_stream_t stream) {
  // everything caote_score would refuse is refused here, before anything touches the stream or the array
  int rc = score_args_check(p, q, K, V, len, base, o, scores);
  if (rc) return rc;
  if (workspace_bytes(p) > kStaticScratchBytes) return CAOTE_ERR_TOO_LARGE;
  rc = check_device();
  if (rc) return rc;
  char* scratch = nullptr;
  rc = static_scratch_address(&scratch);  // first call on this device: looks the address up
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  // the array keeps whatever the previous call left: the status word has to start at zero
  CAOTE_CUDA(cudaMemsetAsync(scratch, 0, kHeaderBytes, st));
  // (no second stream here: making one allocates)
  rc = score_impl(p, q, K, V, len, base, nullptr, o, scores, scratch, kStaticScratchBytes, stream, false);
  if (rc) return rc;
  if (status_out) CAOTE_CUDA(cudaMemcpyAsync(status_out, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  return CAOTE_OK;
}

int caote_select_evict(const caote_params_t* p, const float* scores, const int32_t* len, const int32_t* budget,
                       const int32_t* pos, int32_t* evict_idx, int32_t max_evict, int32_t* n_evict,
                       void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  if (!params_ok(p) || !scores || !len || !budget || !evict_idx || !n_evict || !workspace || max_evict < 1)
    return CAOTE_ERR_INVALID_ARG;
  if (workspace_bytes_ < kHeaderBytes || !aligned(workspace, 256)) return CAOTE_ERR_INVALID_ARG;
  int rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  cudaStream_t st = (cudaStream_t)stream;
  CAOTE_LAUNCH("select_kernel", st, launch_pdl(sel::select_kernel, dim3(dm.units), dim3(sel::kSelThreads), 0, st, 
      dm.Hkv, dm.cap, scores, len, budget, pos, evict_idx, max_evict, n_evict, (int*)workspace));
  return CAOTE_OK;
}

int caote_select_evict_greedy(const caote_params_t* p, const void* V, const float* h, const int32_t* len,
                              const int32_t* budget, const int32_t* pos, int32_t* evict_idx, int32_t* order,
                              int32_t max_evict, int32_t* n_evict, void* workspace, size_t workspace_bytes_,
                              caote_stream_t stream) {
  if (!params_ok(p) || !V || !h || !len || !budget || !evict_idx || !n_evict || !workspace || max_evict < 1)
    return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p) || p->capacity > greedy::kMaxTokens) return CAOTE_ERR_UNSUPPORTED;
  if (workspace_bytes_ < kHeaderBytes || !aligned(workspace, 256) || !aligned(V, 16)) return CAOTE_ERR_INVALID_ARG;
  int rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  cudaStream_t st = (cudaStream_t)stream;
  int* status = (int*)workspace;
  if (p->dtype == CAOTE_BF16) {
    if (dm.D == 128) {
      bool used = false;
      rc = launch_greedy_cluster(dm, V, h, len, budget, pos, evict_idx, order, max_evict, n_evict, status, st, &used);
      if (rc || used) return rc;
      return launch_greedy<__nv_bfloat16, 128>(dm, V, h, len, budget, pos, evict_idx, order, max_evict, n_evict, status, st);
    }
    return launch_greedy<__nv_bfloat16, 64>(dm, V, h, len, budget, pos, evict_idx, order, max_evict, n_evict, status, st);
  }
  if (dm.D == 128) return launch_greedy<float, 128>(dm, V, h, len, budget, pos, evict_idx, order, max_evict, n_evict, status, st);
  return launch_greedy<float, 64>(dm, V, h, len, budget, pos, evict_idx, order, max_evict, n_evict, status, st);
}

int caote_compact(const caote_params_t* p, void* K, void* V, float* base, int32_t* pos, int32_t* len,
                  const int32_t* evict_idx, int32_t max_evict, const int32_t* n_evict, int32_t mode,
                  void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  if (!params_ok(p) || !K || !V || !len || !evict_idx || !n_evict || !workspace || max_evict < 1)
    return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  if (mode != CAOTE_COMPACT_FILL && mode != CAOTE_COMPACT_STABLE) return CAOTE_ERR_INVALID_ARG;
  if (workspace_bytes_ < kHeaderBytes || !aligned(workspace, 256)) return CAOTE_ERR_INVALID_ARG;
  if (!aligned(K, 16) || !aligned(V, 16)) return CAOTE_ERR_INVALID_ARG;
  int rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  const int row_bytes = dm.D * (p->dtype == CAOTE_BF16 ? 2 : 4);
  cudaStream_t st = (cudaStream_t)stream;
  if (mode == CAOTE_COMPACT_FILL) {
    CAOTE_LAUNCH("compact_fill_kernel", st, launch_pdl(sel::compact_fill_kernel, dim3(dm.units), dim3(256), 0, st, dm.Hkv, dm.cap, row_bytes, (char*)K, (char*)V, base, pos,
                                                       len, evict_idx, max_evict, n_evict));
  } else {
    dim3 grid(dm.units, 3);
    CAOTE_LAUNCH("compact_stable_kernel", st, sel::compact_stable_kernel<<<grid, 256, (size_t)sel::kStableTile * row_bytes, st>>>(
        dm.Hkv, dm.cap, row_bytes, (char*)K, (char*)V, base, pos, len, evict_idx, max_evict, n_evict));
  }
  CAOTE_LAUNCH("update_len_kernel", st, launch_pdl(sel::update_len_kernel, dim3((dm.B + 127) / 128), dim3(128), 0, st, dm.B, len, n_evict));
  return CAOTE_OK;
}

// caote_step (vsum == NULL) and caote_step_fast (vsum kept current: += appended rows, -= evicted rows).
static int step_impl(const caote_params_t* p, const void* q, const void* k_new, const void* v_new, void* K, void* V,
                     float* base, int32_t* pos, int32_t* len, int32_t* n_seen, const int32_t* budget, float* vsum,
                     float* o, float* scores, int32_t* evict_idx, int32_t max_evict, int32_t* n_evict,
                     int32_t compact_mode, void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  // every host-visible check of the calls below runs before the first launch
  int rc = score_args_check(p, q, K, V, len, base, o, scores);
  if (!rc) rc = score_workspace_check(p, workspace, workspace_bytes_);
  if (!rc && (k_new || v_new)) rc = append_args_check(p, K, V, len, k_new, v_new, workspace, workspace_bytes_);
  if (!rc && (!budget || !evict_idx || !n_evict || max_evict < 1)) rc = CAOTE_ERR_INVALID_ARG;
  if (!rc && compact_mode != CAOTE_COMPACT_FILL && compact_mode != CAOTE_COMPACT_STABLE) rc = CAOTE_ERR_INVALID_ARG;
  if (!rc) rc = check_device();
  if (rc) return rc;
  const bool bf16 = p->dtype == CAOTE_BF16;
  if (k_new || v_new) {
    const Dims dma = make_dims(p);
    const bool fold = vsum && dma.m == 1 && append_per_sequence(dma);  // the append adds the new value rows itself
    if (vsum && !fold) {
      const Dims dm = make_dims(p);
      cudaStream_t st = (cudaStream_t)stream;
      if (bf16) {
        CAOTE_LAUNCH("fast_vsum_add_kernel", st, fast::vsum_add_kernel<__nv_bfloat16><<<dm.units, dm.D, 0, st>>>(
            dm.Hkv, dm.cap, dm.m, dm.D, (const __nv_bfloat16*)v_new, len, vsum));
      } else {
        CAOTE_LAUNCH("fast_vsum_add_kernel", st, fast::vsum_add_kernel<float><<<dm.units, dm.D, 0, st>>>(
            dm.Hkv, dm.cap, dm.m, dm.D, (const float*)v_new, len, vsum));
      }
    }
    rc = append_impl(p, K, V, base, pos, len, n_seen, k_new, v_new, workspace, workspace_bytes_, stream,
                     fold ? vsum : nullptr);
    if (rc) return rc;
  }
  rc = score_impl(p, q, K, V, len, base, vsum, o, scores, workspace, workspace_bytes_, stream);
  if (rc) return rc;
  if (compact_mode == CAOTE_COMPACT_FILL) {
    // selection, compaction and the length update in one launch (same results as the two calls below)
    if (!budget || !evict_idx || !n_evict || max_evict < 1) return CAOTE_ERR_INVALID_ARG;
    const Dims dm = make_dims(p);
    const int row_bytes = dm.D * (p->dtype == CAOTE_BF16 ? 2 : 4);
    cudaStream_t st = (cudaStream_t)stream;
    int* hdr = reinterpret_cast<int*>(workspace);
    CAOTE_LAUNCH("select_compact_kernel", st,
                 launch_pdl(sel::select_compact_kernel, dim3(dm.units), dim3(sel::kSelThreads), 0, st, 
                     dm.B, dm.Hkv, dm.cap, row_bytes, scores, (char*)K, (char*)V, base, pos, len, budget, evict_idx,
                     max_evict, n_evict, hdr, hdr + 4, vsum, bf16 ? 2 : 4));
    return CAOTE_OK;
  }
  rc = caote_select_evict(p, scores, len, budget, pos, evict_idx, max_evict, n_evict, workspace,
                          workspace_bytes_, stream);
  if (rc) return rc;
  if (vsum) {
    const Dims dm = make_dims(p);
    cudaStream_t st = (cudaStream_t)stream;
    if (bf16) {
      CAOTE_LAUNCH("fast_vsum_sub_kernel", st, fast::vsum_sub_kernel<__nv_bfloat16><<<dm.units, 128, 0, st>>>(
          dm.Hkv, dm.cap, dm.D, (const __nv_bfloat16*)V, evict_idx, max_evict, n_evict, vsum));
    } else {
      CAOTE_LAUNCH("fast_vsum_sub_kernel", st, fast::vsum_sub_kernel<float><<<dm.units, 128, 0, st>>>(
          dm.Hkv, dm.cap, dm.D, (const float*)V, evict_idx, max_evict, n_evict, vsum));
    }
  }
  return caote_compact(p, K, V, base, pos, len, evict_idx, max_evict, n_evict, compact_mode, workspace,
                       workspace_bytes_, stream);
}

int caote_step(const caote_params_t* p, const void* q, const void* k_new, const void* v_new, void* K, void* V,
               float* base, int32_t* pos, int32_t* len, int32_t* n_seen, const int32_t* budget, float* o,
               float* scores, int32_t* evict_idx, int32_t max_evict, int32_t* n_evict, int32_t compact_mode,
               void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  return step_impl(p, q, k_new, v_new, K, V, base, pos, len, n_seen, budget, nullptr, o, scores, evict_idx, max_evict,
                   n_evict, compact_mode, workspace, workspace_bytes_, stream);
}

int caote_step_fast(const caote_params_t* p, const void* q, const void* k_new, const void* v_new, void* K, void* V,
                    float* base, int32_t* pos, int32_t* len, int32_t* n_seen, const int32_t* budget, float* vsum,
                    float* o, float* scores, int32_t* evict_idx, int32_t max_evict, int32_t* n_evict,
                    int32_t compact_mode, void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  if (!vsum || !aligned(vsum, 16)) return CAOTE_ERR_INVALID_ARG;
  return step_impl(p, q, k_new, v_new, K, V, base, pos, len, n_seen, budget, vsum, o, scores, evict_idx, max_evict,
                   n_evict, compact_mode, workspace, workspace_bytes_, stream);
}

static int post_evict_impl(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                           const int32_t* evict_idx, int32_t max_evict, const int32_t* n_evict, const float* o,
                           float* o_post, const char* ws, caote_stream_t stream) {
  if (!params_ok(p) || !q || !K || !V || !len || !evict_idx || !n_evict || !o || !o_post || max_evict < 1)
    return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  if (!aligned(q, 16) || !aligned(K, 16) || !aligned(V, 16)) return CAOTE_ERR_INVALID_ARG;
  int rc = check_device();
  if (rc) return rc;
  const Dims dm = make_dims(p);
  cudaStream_t st = (cudaStream_t)stream;
  if (p->dtype == CAOTE_BF16) {
    if (dm.D == 128) return launch_post_evict<__nv_bfloat16, 128>(dm, q, K, V, len, evict_idx, max_evict, n_evict, o, o_post, ws, st);
    return launch_post_evict<__nv_bfloat16, 64>(dm, q, K, V, len, evict_idx, max_evict, n_evict, o, o_post, ws, st);
  }
  if (dm.D == 128) return launch_post_evict<float, 128>(dm, q, K, V, len, evict_idx, max_evict, n_evict, o, o_post, ws, st);
  return launch_post_evict<float, 64>(dm, q, K, V, len, evict_idx, max_evict, n_evict, o, o_post, ws, st);
}

int caote_post_evict_output(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                            const int32_t* evict_idx, int32_t max_evict, const int32_t* n_evict, const float* o,
                            float* o_post, caote_stream_t stream) {
  return post_evict_impl(p, q, K, V, len, evict_idx, max_evict, n_evict, o, o_post, nullptr, stream);
}

int caote_post_evict_output_ws(const caote_params_t* p, const void* q, const void* K, const void* V, const int32_t* len,
                               const int32_t* evict_idx, int32_t max_evict, const int32_t* n_evict, const float* o,
                               float* o_post, const void* workspace, size_t workspace_bytes_, caote_stream_t stream) {
  if (!params_ok(p)) return CAOTE_ERR_INVALID_ARG;
  if (!params_supported(p)) return CAOTE_ERR_UNSUPPORTED;
  const int rc = score_workspace_check(p, workspace, workspace_bytes_);
  if (rc) return rc;
  return post_evict_impl(p, q, K, V, len, evict_idx, max_evict, n_evict, o, o_post, (const char*)workspace, stream);
}

int caote_read_status(void* workspace, caote_stream_t stream, int32_t* status_out) {
  if (!workspace || !status_out) return CAOTE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  CAOTE_CUDA(cudaMemcpyAsync(status_out, workspace, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  CAOTE_CUDA(cudaMemsetAsync(workspace, 0, sizeof(int32_t), st));
  CAOTE_CUDA(cudaStreamSynchronize(st));
  return CAOTE_OK;
}

const char* caote_status_string(int status) {
  switch (status) {
    case CAOTE_OK: return "ok";
    case CAOTE_ERR_INVALID_ARG: return "invalid argument";
    case CAOTE_ERR_UNSUPPORTED: return "unsupported dtype, head_dim, mode or device";
    case CAOTE_ERR_CUDA: return "CUDA call failed";
    case CAOTE_ERR_TIMEOUT: return "a bounded device-side wait gave up";
    case CAOTE_ERR_BAD_LENGTH: return "a cache length is outside [n_new, capacity]";
    case CAOTE_ERR_OVERFLOW: return "more evictions than max_evict, or an append past capacity";
    case CAOTE_ERR_TOO_LARGE: return "the problem needs more scratch than the built-in array of caote_score_static holds";
    default: return "unknown status";
  }
}

const char* caote_last_cuda_error(void) { return g_cuda_error; }

int caote_trace_enable(int on) {
  g_trace_on.store(on != 0, std::memory_order_relaxed);
  return CAOTE_OK;
}

int caote_trace_collect(caote_trace_entry_t* out, int32_t max_entries, int32_t* n_out) {
  if (!out || !n_out || max_entries < 1) return CAOTE_ERR_INVALID_ARG;
  std::vector<TraceRec> recs;
  {
    std::lock_guard<std::mutex> lk(g_trace_mu);
    recs.swap(g_trace_pending);
  }
  int n = 0;
  int rc = CAOTE_OK;
  for (const TraceRec& r : recs) {
    float ms = 0.f;
    cudaError_t e = cudaEventSynchronize(r.b);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.a, r.b);
    if (e != cudaSuccess) rc = cuda_fail(e, "caote_trace_collect");
    int i = 0;
    for (; i < n; ++i)
      if (strncmp(out[i].name, r.name, sizeof(out[i].name) - 1) == 0) break;
    if (i == n && n < max_entries) {
      memset(&out[n], 0, sizeof(out[n]));
      strncpy(out[n].name, r.name, sizeof(out[n].name) - 1);
      ++n;
    }
    if (i < n && e == cudaSuccess) {
      out[i].launches += 1;
      out[i].total_ms += (double)ms;
    }
    std::lock_guard<std::mutex> lk(g_trace_mu);
    g_trace_pool.push_back(r.a);
    g_trace_pool.push_back(r.b);
  }
  *n_out = n;
  return rc;
}

int caote_set_option(int32_t option, int64_t value) {
  switch (option) {
    case CAOTE_OPT_WAIT_CYCLES:
      if (value < 1) return CAOTE_ERR_INVALID_ARG;
      g_wait_cycles.store((long long)value, std::memory_order_relaxed);
      return CAOTE_OK;
    case CAOTE_OPT_SIDE_BY_SIDE:
      if (value < 0 || value > 1 + 64) return CAOTE_ERR_INVALID_ARG;
      g_side_by_side.store((int)value, std::memory_order_relaxed);
      return CAOTE_OK;
    case CAOTE_OPT_DECODE_CLUSTER:
      if (value < -1 || value > dcl::kMaxC) return CAOTE_ERR_INVALID_ARG;
      g_decode_cluster.store((int)value, std::memory_order_relaxed);
      return CAOTE_OK;
    default:
      return CAOTE_ERR_INVALID_ARG;
  }
}

int64_t caote_launch_count(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
