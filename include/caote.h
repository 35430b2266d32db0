/*
 * caote.h — C ABI of the CAOTE eviction-scoring attention step for NVIDIA B200 (sm_100a).
 *
 * CAOTE ("Cache selection via Attention Output error-based Token Eviction") scores every cached
 * token j of a (sequence, KV head) unit by the change in attention output that evicting it would
 * cause, c_j = w_j / (1 - w_j) * || X - v_j ||_2, keeps the highest-scoring tokens up to a budget
 * and drops the rest from the K/V cache.
 *
 * Conventions shared by every entry point
 * ---------------------------------------
 * Notation (Sec. 2 "Background" and Sec. 3 of the paper): B sequences, Hq query heads, Hkv KV heads,
 * G = Hq / Hkv query heads per KV head (query head hq belongs to KV head hq / G), d = head_dim,
 * cap = slots per unit, n = len[b] valid slots of sequence b (the m = n_new newest tokens included),
 * budget b. A "unit" is one (sequence, KV head) pair; unit index u = b * Hkv + hkv.
 *
 * Layout. All arrays are dense, row-major, innermost dimension last:
 *   q            [B, Hq,  m,   d]   I/O dtype (bf16 or fp32)
 *   K, V         [B, Hkv, cap, d]   I/O dtype; slot j of unit u holds one cached token
 *   o            [B, Hq,  m,   d]   fp32 (the fp32 accumulator is handed out unrounded)
 *   base, scores [B, Hkv, cap]      fp32
 *   pos          [B, Hkv, cap]      int32, original position of the token held by each slot
 *   len, budget, n_evict, n_seen [B] int32
 *   evict_idx    [B, Hkv, max_evict] int32
 * Every pointer named below is a DEVICE pointer unless it says "host". K, V, q, o must be 16-byte
 * aligned; the others 4-byte aligned; workspace 256-byte aligned.
 *
 * Ownership. The caller owns every buffer and the stream. The library allocates no device memory,
 * keeps no per-call state, never synchronises (except caote_read_status) and only enqueues work on
 * the stream it is given. Calls on the same stream compose in order.
 *
 * Errors. Every entry point returns CAOTE_OK (0) or a negative caote_status_t. Arguments that the
 * host can see (null pointers, shapes, workspace size, dtype, head_dim) are validated before any
 * launch and yield CAOTE_ERR_INVALID_ARG / CAOTE_ERR_UNSUPPORTED; nothing is enqueued in that case.
 * Conditions only the device can see (len[b] > cap, len[b] < n_new, more evictions than max_evict,
 * an append that would overflow cap) make the kernel skip that sequence and record a code in the
 * workspace status word, read back with caote_read_status. No entry point throws, aborts or traps.
 */
#ifndef CAOTE_H_
#define CAOTE_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define CAOTE_API __attribute__((visibility("default")))
#else
#define CAOTE_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

/* A CUDA stream handle (cudaStream_t), passed as an opaque pointer so that this header needs no CUDA
 * include. NULL is the legacy default stream. */
typedef void* caote_stream_t;

typedef enum {
  CAOTE_OK = 0,
  CAOTE_ERR_INVALID_ARG = -1, /* null pointer, bad shape, workspace too small                     */
  CAOTE_ERR_UNSUPPORTED = -2, /* dtype / head_dim / mode not built, or the device is not sm_100   */
  CAOTE_ERR_CUDA = -3,        /* a CUDA runtime or driver call failed (see caote_last_cuda_error) */
  CAOTE_ERR_TIMEOUT = -4,     /* a bounded device-side wait gave up (status word only)            */
  CAOTE_ERR_BAD_LENGTH = -5,  /* device saw len[b] > cap or 0 < len[b] < n_new (status word only) */
  CAOTE_ERR_OVERFLOW = -6,    /* device saw n_evict > max_evict or len + n_new > cap (status word) */
  CAOTE_ERR_TOO_LARGE = -7    /* caote_score_static: the shape needs more than CAOTE_STATIC_SCRATCH_BYTES */
} caote_status_t;

typedef enum { CAOTE_BF16 = 0, CAOTE_F32 = 1 } caote_dtype_t;

/* How the base retention score h_j is obtained from the attention matrix A (rows = this call's
 * queries, columns = cached tokens), Sec. 2 (f_score) and Sec. 3.2:
 *   LAST_QUERY  h_j = sum_g A^g[m-1, j]                 (TOVA: the last query row of every group head)
 *   CHUNK_SUM   h_j = sum_g sum_i A^g[i, j]             (H2O over this call's block of m queries only)
 *   ACCUM       base_j += sum_g sum_i A^g[i, j]; h = base   (H2O carried across calls; base is in/out)
 *   EXTERNAL    h_j = base_j                            (any non-negative score the caller computed)
 */
typedef enum {
  CAOTE_BASE_LAST_QUERY = 0,
  CAOTE_BASE_CHUNK_SUM = 1,
  CAOTE_BASE_ACCUM = 2,
  CAOTE_BASE_EXTERNAL = 3
} caote_base_mode_t;

/* How the cache is repacked after eviction.
 *   FILL    surviving tokens of the last k slots move into the holes left below the new length;
 *           at most k rows move per unit; slot order is not position order afterwards (use pos).
 *   STABLE  surviving tokens keep their relative order (everything behind the first hole shifts).
 */
typedef enum { CAOTE_COMPACT_FILL = 0, CAOTE_COMPACT_STABLE = 1 } caote_compact_mode_t;

typedef struct {
  int32_t batch;      /* B >= 1                                                                    */
  int32_t n_q_heads;  /* Hq, a multiple of n_kv_heads; G = Hq / Hkv <= 16                          */
  int32_t n_kv_heads; /* Hkv >= 1                                                                  */
  int32_t head_dim;   /* d in {64, 128}                                                            */
  int32_t capacity;   /* cap: slots per unit in K, V, base, scores, pos                            */
  int32_t n_new;      /* m >= 1: the last m valid slots of every sequence are the keys of this
                         call's own m queries; query i sees slots j <= n - m + i (causal inside
                         the block, Sec. 2 "Block-wise prompt prefill")                            */
  int32_t dtype;      /* caote_dtype_t of q, K, V                                                  */
  float scale;        /* logits are scale * <q, k>; the paper writes Softmax(QK^T) without a scale,
                         callers normally pass 1/sqrt(head_dim)                                    */
  int32_t base_mode;  /* caote_base_mode_t                                                         */
  int32_t flags;      /* reserved, must be 0                                                       */
} caote_params_t;

/* Bytes of scratch that caote_score / caote_select_evict / caote_compact / caote_append need for these
 * parameters (the maximum over the four; one buffer serves all). Returns 0 if params is invalid.
 * The first 256 bytes hold the status word and the library's own counters; zero them once
 * (cudaMemsetAsync) before first use and leave them alone afterwards. */
CAOTE_API size_t caote_workspace_bytes(const caote_params_t* params);

/* Append the m = n_new newest tokens of every sequence to its cache (Sec. 2: the block
 * [K_{:t}, K_{t+1:t+m}] the new queries attend to). For sequence b with n = len[b]:
 * K/V[b, h, n + i, :] = k_new/v_new[b, h, i, :], base[...] = 0, pos[...] = n_seen[b] + i for
 * i in [0, m); then len[b] = n + m and n_seen[b] += m.
 *   k_new, v_new  [B, Hkv, m, d] I/O dtype, in.     base, pos, n_seen: nullable (skipped when NULL).
 * A sequence with n + m > cap is skipped and CAOTE_ERR_OVERFLOW is recorded. */
CAOTE_API int caote_append(const caote_params_t* params, void* K, void* V, float* base, int32_t* pos,
                 int32_t* len, int32_t* n_seen, const void* k_new, const void* v_new,
                 void* workspace, size_t workspace_bytes, caote_stream_t stream);

/* Attention + CAOTE scores for every unit.
 *   1. alpha^g_i = softmax_j(scale * <q^g_i, k_j>) over visible slots j <= n - m + i, and the
 *      pre-eviction attention output o^g_i = sum_j alpha^g_{i,j} v_j   (Sec. 2, generation and
 *      block-wise prefill equations; Sec. 3.1, X_attn = V A^T).
 *   2. base score h per base_mode (Sec. 2 f_score; Sec. 3.2 "CAOTE for H2O"), summed over the G
 *      query heads that share the KV head.
 *   3. w_j = h_j / sum_i h_i (Sec. 3.2, normalisation equation) and X = sum_j w_j v_j.
 *   4. scores[u, j] = w_j / (1 - w_j) * || X - v_j ||_2  (Sec. 3.1 CAOTE score; Sec. 3.2 general
 *      form; Theorem 3.2 shows it equals the output error of evicting j and renormalising).
 *      1 - w_j == 0 gives +inf; sum_i h_i == 0 gives 0. Scores are >= +0 and never NaN for finite
 *      inputs.
 *   q in; K, V in; len in (n = len[b]; 0 skips the sequence; n_new <= n <= cap required);
 *   base: in/out for ACCUM, in for EXTERNAL, ignored (may be NULL) otherwise;
 *   o out (all m rows of all Hq heads); scores out for slots j < n, slots >= n are left untouched. */
CAOTE_API int caote_score(const caote_params_t* params, const void* q, const void* K, const void* V,
                const int32_t* len, float* base, float* o, float* scores, void* workspace,
                size_t workspace_bytes, caote_stream_t stream);

/* caote_score for callers that cannot allocate device memory. (The paper has no counterpart: this is
 * a packaging variant of caote_score, same arithmetic, same kernels.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a serving engine whose memory
 * pool has already claimed the whole GPU, in a plug-in that is handed tensors but no allocator, or on
 * a latency path where an allocation (which may synchronise the device) is not acceptable - and that
 * therefore has nowhere to get the workspace caote_score asks for.
 *
 * Here the scratch is an array of CAOTE_STATIC_SCRATCH_BYTES bytes built into the library's device
 * image; every GPU that loads the library holds it from load until the process exits. The caller
 * passes only inputs and outputs, with the meaning, layout and alignment they have in caote_score.
 *   status_out  device pointer to one int32, or NULL. Receives the status word of this call (CAOTE_OK
 *               or the first device-side error); stream-ordered like the other outputs. Left untouched
 *               when the call itself returns an error code.
 * Limits and rules:
 *   - A shape with caote_workspace_bytes(params) > CAOTE_STATIC_SCRATCH_BYTES is rejected with
 *     CAOTE_ERR_TOO_LARGE, and every argument caote_score would refuse is refused with the same code,
 *     before anything is enqueued or the array is touched.
 *   - The call itself allocates and frees nothing: no cudaMalloc / cudaFree, no allocating library
 *     routine. It enqueues a 256-byte memset of the scratch header, the kernels of caote_score and a
 *     4-byte device-to-device copy.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with
 *     that device current). Make that first call outside any stream capture.
 *   - All calls on one device share the one array, and it keeps the previous call's contents (the call
 *     clears what has to start at zero). Two calls that may overlap on the GPU - different streams
 *     without an ordering between them - race on it and give undefined results; serialise them. */
#define CAOTE_STATIC_SCRATCH_BYTES (16u << 20)
CAOTE_API int caote_score_static(const caote_params_t* params, const void* q, const void* K, const void* V,
                       const int32_t* len, float* base, float* o, float* scores, int32_t* status_out,
                       caote_stream_t stream);

/* Choose the tokens to evict: for sequence b, k = max(0, len[b] - budget[b]) (Sec. 2: the top-b tokens
 * by score are retained; Sec. 4.1 "Prompt consumption": evict once the cache exceeds the budget), and
 * every unit of b evicts its k smallest entries under the total order (score bits, pos) ascending —
 * among equal scores the older token goes first. pos == NULL uses the slot index as pos.
 *   evict_idx[u, 0..k) out: the evicted SLOT indices in ascending order; n_evict[b] = k out.
 * budget[b] >= 1 required (a smaller value is treated as 1). k > max_evict records
 * CAOTE_ERR_OVERFLOW, sets n_evict[b] = 0 and evicts nothing for that sequence. */
CAOTE_API int caote_select_evict(const caote_params_t* params, const float* scores, const int32_t* len,
                       const int32_t* budget, const int32_t* pos, int32_t* evict_idx,
                       int32_t max_evict, int32_t* n_evict, void* workspace,
                       size_t workspace_bytes, caote_stream_t stream);

/* Greedy multi-token eviction (Appendix B, "Extending CAOTE to multi-token eviction": evicting token 1 and then
 * token 2 from the renormalised state, chained): instead of taking the k lowest scores of one scoring pass,
 * evict one token at a time and let every eviction change the scores of the rest. Per unit, with
 * non-negative weights h_j (any base score: accumulated H2O scores after caote_score, or scores of the
 * caller's own), w_j = h_j / sum_i h_i and X = sum_j w_j v_j, repeat k = max(0, len - budget) times:
 *     e = arg min_j  w_j / (1 - w_j) * || X - v_j ||_2   over the tokens still present (ties: smaller pos),
 *     X <- (X - w_e v_e) / (1 - w_e),   w_i <- w_i / (1 - w_e)   (the paper's alpha' and X').
 * After t evictions the distance between the original and the current X is the paper's closed-form joint
 * score of the evicted set. With k = 1 the result is that of caote_select_evict on the CAOTE scores.
 *   V [B, Hkv, cap, d] I/O dtype, in;  h [B, Hkv, cap] fp32, in (negative values count as 0);
 *   evict_idx[u, 0..k) out: the evicted slots in ascending order (what caote_compact takes);
 *   order[u, 0..k) out, nullable: the same slots in the order they were evicted;  n_evict[b] = k out.
 * capacity <= 24576 (the unit's weights and distances stay in shared memory), else CAOTE_ERR_UNSUPPORTED.
 * Cost: one sweep over the unit's value rows per eviction (from L2 after the first). */
CAOTE_API int caote_select_evict_greedy(const caote_params_t* params, const void* V, const float* h,
                              const int32_t* len, const int32_t* budget, const int32_t* pos,
                              int32_t* evict_idx, int32_t* order, int32_t max_evict, int32_t* n_evict,
                              void* workspace, size_t workspace_bytes, caote_stream_t stream);

/* Remove the evicted slots from K, V, base, pos in place and set len[b] -= n_evict[b], so that the
 * cache is back within budget before the next block arrives (Sec. 2, budgeted block-wise flow).
 * mode is a caote_compact_mode_t. base, pos nullable. evict_idx rows must be ascending and unique
 * (what caote_select_evict writes). */
CAOTE_API int caote_compact(const caote_params_t* params, void* K, void* V, float* base, int32_t* pos,
                  int32_t* len, const int32_t* evict_idx, int32_t max_evict, const int32_t* n_evict,
                  int32_t mode, void* workspace, size_t workspace_bytes, caote_stream_t stream);

/* One whole eviction step on the stream: caote_append (skipped when k_new is NULL), caote_score,
 * caote_select_evict, caote_compact, with the same arguments and the same results as the four
 * separate calls. */
CAOTE_API int caote_step(const caote_params_t* params, const void* q, const void* k_new, const void* v_new,
               void* K, void* V, float* base, int32_t* pos, int32_t* len, int32_t* n_seen,
               const int32_t* budget, float* o, float* scores, int32_t* evict_idx, int32_t max_evict,
               int32_t* n_evict, int32_t compact_mode, void* workspace, size_t workspace_bytes,
               caote_stream_t stream);

/* ---- FastCAOTE (Sec. 3.3) ------------------------------------------------------------------------
 * The same score with the pre-eviction output replaced by the plain mean of the cached values:
 *     c_j = w_j / (1 - w_j) * || (1/n) sum_i v_i - v_j ||_2 ,
 * everything else (attention, o, base score per base_mode, normalisation, selection) as in caote_score.
 * The mean does not depend on the current queries, so it is carried from step to step instead of being
 * recomputed: vsum [B, Hkv, d] fp32 holds, per unit, the sum of its n valid V rows (new tokens
 * included). On the single-query path this removes the second pass over V: K and V are read once. */

/* vsum[u, :] = sum_{j < len} V[u, j, :] from scratch (one read of V); len 0 gives 0. */
CAOTE_API int caote_vsum(const caote_params_t* params, const void* V, const int32_t* len, float* vsum,
               caote_stream_t stream);

/* caote_score with FastCAOTE scores. vsum: in, current for the cache as passed (16-byte aligned). */
CAOTE_API int caote_score_fast(const caote_params_t* params, const void* q, const void* K, const void* V,
                     const int32_t* len, float* base, const float* vsum, float* o, float* scores,
                     void* workspace, size_t workspace_bytes, caote_stream_t stream);

/* caote_step with FastCAOTE scores. vsum: in/out; the rows appended by this call are added before
 * scoring and the rows it evicts are subtracted, so that it is current for the next call. Sums are kept
 * in fp32: refresh with caote_vsum now and then over very long runs if the drift matters. */
CAOTE_API int caote_step_fast(const caote_params_t* params, const void* q, const void* k_new, const void* v_new,
                    void* K, void* V, float* base, int32_t* pos, int32_t* len, int32_t* n_seen,
                    const int32_t* budget, float* vsum, float* o, float* scores, int32_t* evict_idx,
                    int32_t max_evict, int32_t* n_evict, int32_t compact_mode, void* workspace,
                    size_t workspace_bytes, caote_stream_t stream);

/* caote_score with the other way of extending the single-head, single-query score to a group of query
 * heads and to a block of queries: instead of adding the rows' attention weights and applying the general
 * form once per unit, add up the exact single-query errors (Sec. 3.1 score, Theorem 3.2, row by row) of
 * the rows that define the base score,
 *     scores[u, j] = sum_r alpha_{r,j} / (1 - alpha_{r,j}) * || o_r - v_j ||_2 ,
 * r over the last row of every group head (LAST_QUERY) or over all rows (CHUNK_SUM); other base modes
 * return CAOTE_ERR_UNSUPPORTED. With one head and one query it equals caote_score. Arguments as in
 * caote_score (no base). Runs on the any-shape fp32 CUDA-core kernels (two dot products of length d per
 * (row, token) pair): a correctness path for comparing the two aggregations, not tuned. */
CAOTE_API int caote_score_sum_errors(const caote_params_t* params, const void* q, const void* K, const void* V,
                           const int32_t* len, float* o, float* scores, void* workspace,
                           size_t workspace_bytes, caote_stream_t stream);

/* Post-eviction attention output (Sec. 2: the budgeted cache attends over the retained tokens only;
 * Sec. 3.1, proof of Theorem 3.2): for every query row r of this call,
 *     o_post_r = (o_r - sum_{e in E_r} alpha_{r,e} v_e) / (1 - sum_{e in E_r} alpha_{r,e}),
 * E_r = the evicted slots row r can see, alpha = the row's pre-eviction softmax weights; i.e. the softmax
 * attention over the retained tokens. A row whose visible tokens are all evicted gets 0.
 * Call it after caote_select_evict and BEFORE caote_compact (evict_idx refers to the slots as scored):
 *   q, K, V, len as passed to caote_score; evict_idx, max_evict, n_evict as written by caote_select_evict;
 *   o  in:  the pre-eviction output caote_score wrote, [B, Hq, m, d] fp32;
 *   o_post out, same shape (may alias o).
 * Needs no workspace. It recomputes the rows' softmax normalisers with one pass over K on the CUDA cores;
 * caote_post_evict_output_ws below avoids that pass where it can. */
CAOTE_API int caote_post_evict_output(const caote_params_t* params, const void* q, const void* K, const void* V,
                            const int32_t* len, const int32_t* evict_idx, int32_t max_evict,
                            const int32_t* n_evict, const float* o, float* o_post, caote_stream_t stream);

/* The same result from the softmax statistics that scoring already produced (Sec. 3.1: the weights
 * alpha_{r,e} of the evicted tokens are all the correction needs): `workspace` is the one the caote_score /
 * caote_step... call that scored these slots ran on, with the same params, and nothing else has run on it
 * since except caote_select_evict[_greedy]. The tensor-core kernels (single-query decode on thread-block
 * clusters; chunked prefill) leave every row's log-sum-exp there and say so in the workspace header; this
 * call then reads q, o and only the evicted K / V rows, which makes it a small fraction of a scoring call.
 * After any other scoring path the header says "none" and the call does what caote_post_evict_output does.
 * Arguments as above; workspace (device, 256-byte aligned) of at least caote_workspace_bytes(params),
 * read only. Errors as above, and CAOTE_ERR_INVALID_ARG for a missing, short or misaligned workspace. */
CAOTE_API int caote_post_evict_output_ws(const caote_params_t* params, const void* q, const void* K, const void* V,
                               const int32_t* len, const int32_t* evict_idx, int32_t max_evict,
                               const int32_t* n_evict, const float* o, float* o_post, const void* workspace,
                               size_t workspace_bytes, caote_stream_t stream);

/* Synchronise the stream, copy the status word to *status_out (host pointer) and reset it to CAOTE_OK.
 * The word holds the first device-side error since the last reset. */
CAOTE_API int caote_read_status(void* workspace, caote_stream_t stream, int32_t* status_out);

/* Static, NUL-terminated description of a status code. */
CAOTE_API const char* caote_status_string(int status);

/* Text of the last CUDA error seen by the calling thread inside this library ("" if none). */
CAOTE_API const char* caote_last_cuda_error(void);

/* Per-kernel timing, for benchmarks and profiling. While tracing is on (process-wide switch), every
 * kernel launch of this library is bracketed by two CUDA events recorded on the launching stream.
 * caote_trace_collect waits for the outstanding events, adds up launches and elapsed milliseconds per
 * kernel name into out[0..*n_out) (host memory, at most max_entries names) and forgets them.
 * Do not enable tracing while a stream is being captured into a CUDA graph. */
typedef struct {
  char name[48];
  int64_t launches;
  double total_ms;
} caote_trace_entry_t;
CAOTE_API int caote_trace_enable(int on);
CAOTE_API int caote_trace_collect(caote_trace_entry_t* out, int32_t max_entries, int32_t* n_out);

/* Process-wide settings, for tests and tuning runs. (The paper has no counterpart.)
 *   CAOTE_OPT_WAIT_CYCLES     clock cycles after which a device-side wait of the single-query cluster kernel
 *                             gives up (default 2e9, about a second). The kernel then records
 *                             CAOTE_ERR_TIMEOUT in the status word and still returns; its outputs are
 *                             undefined, the caches and the workspace stay usable. value >= 1.
 *   CAOTE_OPT_DECODE_CLUSTER  CTAs per thread-block cluster on the single-query path: 0 = chosen from the
 *                             shape (default), 1..16 = forced (shapes it cannot serve take the next path),
 *                             -1 = do not use the cluster kernel.
 *   CAOTE_OPT_SIDE_BY_SIDE    1 (default): on the single-query path, when the clusters leave enough SMs idle and
 *                             the units do not divide evenly among them, the last sequences of the batch are
 *                             scored by the streaming kernel on a second stream of the library's own, beside the
 *                             cluster kernel; the caller's stream waits for both. 0 = never. 2..65 = always,
 *                             with the last value - 1 sequences on the streaming kernel (tests, tuning). (The second stream
 *                             and two events are created on first use, one set per device; caote_score_static
 *                             never uses them.)
 * Takes effect for launches made after the call. Returns CAOTE_ERR_INVALID_ARG for an unknown option or a
 * value out of range. */
typedef enum { CAOTE_OPT_WAIT_CYCLES = 1, CAOTE_OPT_DECODE_CLUSTER = 2, CAOTE_OPT_SIDE_BY_SIDE = 3 } caote_option_t;
CAOTE_API int caote_set_option(int32_t option, int64_t value);

/* Number of kernels this library has launched from this process since it was loaded. */
CAOTE_API int64_t caote_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* CAOTE_H_ */
