/*
 * prhs.h -- C ABI of the B200 sparse decode-attention library for Pre-hoc Sparsity
 * (PrHS) with Clustered Indices Sharing (CIS).
 *
 * One decode step of one layer has three parts:
 *   1. retrieval (first step of a block, first layer of a layer group only): score the
 *      query against every cached key and select the exact top-k over the middle range;
 *   2. index-set builder: sinks U (shared, dilated) middle set U recency window;
 *   3. gathered split-K flash-decoding attention over the selected K/V rows only.
 * A dropped-mass diagnostic (delta) reports how much softmax mass the selection lost.
 *
 * Conventions
 *   - Positions are 0-based.  t_b = seq_lens[b] is the number of cached positions visible
 *     to sequence b's current query, the current token (position t_b - 1) included.
 *     sinks = [0, S0), middle candidates = [S0, t - W), local window = [t - W, t).
 *   - head_dim is 128.  q, K, V and attention outputs are bf16; logits, log-sum-exps and
 *     delta are fp32; indices and counts are int32.
 *   - Query head h uses KV head h / (num_q_heads / num_kv_heads).  Index sets are per
 *     (sequence, query head), as in the paper; PRHS_GROUP_SETS is a labelled variant with one
 *     set per (sequence, KV head).
 *   - "device" pointers are CUDA device memory owned by the caller unless stated; "host"
 *     pointers are ordinary (preferably pinned) host memory.  The library never frees or
 *     keeps caller memory beyond the call (asynchronous work on `stream` excepted).
 *   - Every call validates its arguments on the host and returns a prhs_status; nothing
 *     traps or asserts on the device, no kernel waits on another kernel or CTA, and the only
 *     waits there are (on the copy engine's barriers) are bounded.  Device-side anomalies (an
 *     index outside [0, t_b), a page id outside the pool, a wait that ran out) are recorded in
 *     a flag word read by prhs_check().
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*; NULL = the default
 *     stream) and is asynchronous unless stated.  Workspaces and the shared-set state are
 *     allocated in prhs_create(); no call below allocates.
 *   - A context must be used from one host thread at a time and on one stream at a time.
 */
#ifndef PRHS_H_
#define PRHS_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct prhs_ctx prhs_ctx;

typedef enum {
  PRHS_OK = 0,
  PRHS_ERR_INVALID_ARG = 1, /* NULL pointer, bad shape, value out of the configured range */
  PRHS_ERR_UNSUPPORTED = 2, /* head_dim != 128, page_size not in {0,16}, group size > 16   */
  PRHS_ERR_OOM = 3,         /* prhs_create could not allocate its workspaces               */
  PRHS_ERR_CUDA = 4,        /* a CUDA runtime call failed; see prhs_last_error             */
  PRHS_ERR_STATE = 5,       /* no shared set for this block/group (leader not called yet)   */
  PRHS_ERR_CAPACITY = 6,    /* batch, k, window, ... exceed what prhs_create was given      */
  PRHS_ERR_DEVICE_FLAG = 7  /* prhs_check: a kernel recorded an anomaly                    */
} prhs_status;

/* Sizes fixed at prhs_create(); workspaces are dimensioned from them. */
typedef struct {
  int32_t num_layers;    /* layers whose shared sets are kept (groups = ceil(L / layer_group)) */
  int32_t max_batch;     /* B */
  int32_t num_q_heads;   /* Hq */
  int32_t num_kv_heads;  /* Hkv, divides Hq; Hq / Hkv <= 16 */
  int32_t head_dim;      /* must be 128 */
  int32_t max_context;   /* largest t_b ever passed (cache capacity in positions), <= 2^20 */
  int32_t page_size;     /* 0 = contiguous cache, 16 = paged cache */
  int32_t max_k;         /* largest middle budget k */
  int32_t max_window;    /* largest recency window W */
  int32_t max_sinks;     /* largest sink count S0 */
  int32_t max_dilate_r;  /* largest dilation radius r */
  int32_t max_dilate_m;  /* largest number of dilated winners m; -1 = floor(max_k / 3) */
  int32_t min_layer_group; /* smallest layer_group that will be used (sizes the state); >= 1 */
  int32_t max_block_sets;  /* sets kept per (b, h) and block, 1..64; 1 unless the cosine gate is
                              used, which needs max_block_sets >= refresh_interval              */
  uint32_t flags;          /* PRHS_CFG_* below; 0 = defaults                                    */
} prhs_config;

/* Configuration flags */
#define PRHS_CFG_NO_TMA 1u /* retrieval scoring never uses the tensor-memory-accelerator kernels: the
                              key stream is staged by the cp.async ring kernel (mma.sync) instead, which is what
                              the library falls back to on its own when the driver does not export
                              cuTensorMapEncodeTiled or the cache spans 2^31 rows or more.  Same
                              results; for testing that path and for comparing the two. */
#define PRHS_CFG_TMA_GATHER 2u /* the gathered attention (per-head sets) brings its rows in with TMA row
                              gathers (cp.async.bulk.tensor tile::gather4, four rows per instruction,
                              no multicast) instead of 16-byte cp.async copies.  Same results.  Off by
                              default because it measured slower: a tile that ldmatrix reads without
                              bank conflicts needs the 128-byte swizzle, hence two 64-column boxes per
                              row, and at that granularity the copy engine falls behind (a sharing step
                              of the 32K-context layer at batch 8: 49.0 us against 44.1 us).  Kept so
                              that the comparison can be repeated
                              (python -m paper_2602_08329_b200.gather_ceiling). */
#define PRHS_CFG_MMA_SYNC_SCORE 4u /* retrieval scoring runs its contraction with mma.sync in eight
                              consumer warps (score_tma_kernel) instead of on the tcgen05 tensor cores
                              (score_umma_kernel: 128-key tiles staged by TMA, one thread issues the
                              MMAs, accumulators in tensor memory), which is the default.  Same results
                              up to the summation order inside the tensor core; both are bound by the
                              key stream and measure within 1 % of each other.  For testing that
                              kernel and for comparing the two.  Cosine-gated steps use this kernel
                              whatever the flag says: most of their CTAs return at once, and an empty CTA
                              of a kernel that uses tensor memory is several times as expensive. */
#define PRHS_CFG_GROUP_TCGEN05 8u /* the gathered attention of the group-shared variant (PRHS_GROUP_SETS)
                              runs on the tcgen05 tensor cores (gather_group_attn_umma_kernel: 128-row
                              tiles gathered into swizzled shared memory, S and O^T in tensor memory)
                              instead of mma.sync with register accumulators.  Same results up to
                              summation order.  Off by default because it measured slower (sharing step
                              of the variant at 32K, batch 16: 44.5 us against 42.6 us; at 128K, batch 4:
                              40.3 against 34.3; ragged paged batch of 64: 128 against 120): its rings
                              of 128-row tiles leave room for one deep or two shallow CTAs per SM,
                              where the mma.sync kernel pipelines 16-row stages per warp.  Kept for the
                              comparison. */

/* A view of one layer's KV cache (device memory, bf16, caller-owned).
 *   contiguous (page_table == NULL): row i of (b, kvh) is at
 *        k + b*stride_outer + kvh*stride_head + i*128            (element offsets)
 *   paged (page_table != NULL, 16 positions per page): row i of (b, kvh) is at
 *        k + page_table[b*page_table_stride + i/16]*stride_outer + kvh*stride_head + (i%16)*128
 * Rows are 128 contiguous bf16 (256 bytes); k and v must be 16-byte aligned and both strides
 * multiples of 128 elements (whole rows), with fewer than 2^32 rows between the base and the
 * last row addressed. */
typedef struct {
  const void* k;
  const void* v;
  int64_t stride_outer;
  int64_t stride_head;
  const int32_t* page_table; /* device [B][page_table_stride] or NULL */
  int32_t page_table_stride;
  const int32_t* seq_lens;   /* device [B]: t_b, current token included; 0 <= t_b <= max_seq_len */
  int32_t max_seq_len;       /* host-side upper bound of every t_b (sizes the launch); 0 = max_context.
                                The cache must hold max_seq_len positions per (b, kvh): tiled copies
                                may read rows in [t_b, max_seq_len) and ignore them */
  int32_t num_pages;         /* paged: pages in the pool (bounds check); contiguous: ignored */
} prhs_kv_view;

/* Schedule flags */
#define PRHS_DILATE_ANCHOR 1u /* the retrieving (layer, step) also attends over the dilated set */
#define PRHS_WANT_DELTA    2u /* prhs_decode_step fills out_delta (runs a dense log-sum-exp pass
                                 on every non-retrieving call: diagnostic, not the timed path)  */
#define PRHS_GROUP_SETS    4u /* labelled variant, NOT in the paper (its sets are per head, Sec. 4.1):
                                 the query heads that share a KV head share ONE index set.  A position
                                 is ranked by the largest fp32 logit any head of the group gives it;
                                 top-k, dilation and the set follow as for a single head; a gathered
                                 K/V row then serves the whole group.  Outputs keep their [B][Hq]
                                 shapes (the heads of a group receive the same set).  Not combinable
                                 with the cosine gate (PRHS_ERR_UNSUPPORTED).  No effect when
                                 num_q_heads == num_kv_heads. */

/* The knobs of CIS (Sec. 4.1; defaults Sec. 5.1) plus the cross-layer group size. */
typedef struct {
  int32_t refresh_interval;     /* s: block size in decode steps; step % s == 0 retrieves; >= 1 */
  int32_t layer_group;          /* G_L: layers [g*G_L, (g+1)*G_L) reuse layer g*G_L's set; 1 = off */
  int32_t top_k;                /* k: middle budget; ignored where top_k_per_seq != NULL        */
  const int32_t* top_k_per_seq; /* device [B] or NULL; every entry <= max_k                     */
  int32_t window;               /* W = C_local */
  int32_t sinks;                /* S0 = C_sink */
  int32_t dilate_r;             /* r of Eq. 10 */
  int32_t dilate_m;             /* m of Eq. 10; -1 = floor(k / 3) per sequence                  */
  uint32_t flags;
  /* Progressive sliding attention window in decode (Sec. 4.2, Eq. 11): for the paper's layer
   * number l = layer + 1 >= l_s, positions [S0, P) with P = floor((1 - phi^(alpha (l - l_s) /
   * (N - l_s))) t_b) are masked: they are neither retrieval candidates nor attended (sinks
   * stay).  N = prhs_config.num_layers.  psaw_layer_start = l_s (1-based); 0 = off. */
  float psaw_phi;               /* phi in (0, 1); default 0.7 (Sec. 5.1)                        */
  float psaw_alpha;             /* alpha >= 0; default 1                                        */
  int32_t psaw_layer_start;     /* l_s; default floor(3 N / 4); 0 disables the window           */
  /* Cosine gate of CIS (Sec. 4.1 "Similarity Criteria", Eq. 9).  With sim_threshold = tau > -1
   * a step that is not the first of its block shares, per head, the set used by the MOST RECENT
   * earlier step of the block whose query has cosine similarity > tau with the current query,
   * and retrieves a new set only if there is none (paper default tau = 0.8).  The decision is
   * taken on the device by the group's first layer; the other layers of the group follow it.
   * Within a block the steps must then be run in order.  sim_threshold <= -1: gate off, every
   * step of a block shares the block's first set (the fixed schedule). */
  float sim_threshold;
} prhs_schedule;

/* Create / destroy a context on the current CUDA device.  prhs_create allocates every
 * workspace (scores, split-K partials, index lists) and the shared-set state; it returns
 * PRHS_ERR_OOM and leaves *out NULL if the device cannot hold them.  Synchronous. */
prhs_status prhs_create(const prhs_config* cfg, prhs_ctx** out);
prhs_status prhs_destroy(prhs_ctx* ctx);

/* Retrieval pass (Sec. 2.3 "Top-k Oracle"; Sec. 4.1 "Selection Criteria"; Eq. 10).
 * For every (b, h): logits a_i = q_h . k_i / sqrt(128) over i < t_b (Eq. 2); S* = the
 * min(k_b, t_b - W - S0) middle candidates of largest logit, ordered by descending logit,
 * equal logits by ascending position; S^ = S* U { p + j : p among the first m of S*,
 * |j| <= r } clipped to [0, t_b).  S* and S^ are stored in the context as the shared set
 * of `layer`'s group, anchored at `step`.
 *   q            device bf16 [batch][Hq][128]
 *   out_idx      device int32 [batch][Hq][max_k] or NULL: S* in descending-logit order,
 *                entries past the count are -1
 *   out_count    device int32 [batch][Hq] or NULL: |S*|
 *   out_lse_full device fp32 [batch][Hq] or NULL: log sum_{i<t_b} exp(a_i)
 * `layer` must be the first layer of its group. */
prhs_status prhs_score_topk(prhs_ctx* ctx, int32_t layer, int32_t step, const void* q,
                            const prhs_kv_view* kv, const prhs_schedule* sched, int32_t batch,
                            int32_t* out_idx, int32_t* out_count, float* out_lse_full,
                            void* stream);

/* Index-set builder (Sec. 4.1: C_t = sinks U middle U local; Def. 3.2 key-value sharing).
 * C = [0, min(S0,t)) U M U [max(0,t-W), t) at the CURRENT t_b, ascending and unique, where
 * M = S* if (layer, step) is the retrieving call itself and PRHS_DILATE_ANCHOR is off,
 * else M = S^ of the group's anchor.  PRHS_ERR_STATE if the group has no set anchored at
 * step - step % s.
 *   out_idx   device int32 [batch][Hq][idx_stride], idx_stride >= prhs_index_capacity()
 *   out_count device int32 [batch][Hq] */
prhs_status prhs_build_index_set(prhs_ctx* ctx, int32_t layer, int32_t step,
                                 const prhs_schedule* sched, const prhs_kv_view* kv, int32_t batch,
                                 int32_t* out_idx, int32_t idx_stride, int32_t* out_count,
                                 void* stream);

/* Token-sparse attention (Def. 3.1): for every (b, h), softmax attention of q_h restricted
 * to the rows idx[b][h][0..count) of the cache and renormalised over them, computed as
 * split-K online softmax followed by a merge.
 *   idx      device int32 [batch][Hq][idx_stride], each entry in [0, t_b); order is free,
 *            ascending order gathers fastest; duplicates are attended twice
 *   count    device int32 [batch][Hq]; 0 gives a zero output row and lse = -inf
 *   out      device bf16 [batch][Hq][128]
 *   out_lse  device fp32 [batch][Hq] or NULL: log sum_{i in C} exp(a_i)
 * An index outside [0, t_b) is skipped and recorded in the device flag word. */
prhs_status prhs_sparse_decode_attn(prhs_ctx* ctx, const void* q, const prhs_kv_view* kv,
                                    const int32_t* idx, const int32_t* count, int32_t idx_stride,
                                    int32_t batch, void* out, float* out_lse, void* stream);

/* prhs_sparse_decode_attn for callers that cannot allocate device memory.
 * (The paper has no counterpart; this is an integration aid.)
 * Some hosts of this library run where cudaMalloc is off limits: inside a framework that
 * owns the whole device heap and hands out fixed arenas, in a process whose memory budget is
 * frozen after start-up, or between the capture of other work where an allocation would
 * synchronise the device.  They cannot call prhs_create, which allocates the workspaces.
 * This entry point needs no context and calls no cudaMalloc, cudaFree or other allocating
 * routine: the split-K partials, the merge tickets and the anomaly word live in a
 * file-scope device array inside the library (about 4.3 MB, held by every GPU that loads
 * the library until the process exits).  The caller still owns and passes every input and
 * output.
 *   - Limits: batch * num_q_heads <= PRHS_NOALLOC_MAX_UNITS; head_dim 128; contiguous or
 *     paged views as for the other calls.  Larger shapes return PRHS_ERR_CAPACITY.
 *   - The first call on a device looks up the array's device address and sets the kernel's
 *     shared-memory attribute (no allocation); make that first call outside any stream
 *     capture.
 *   - All calls on a device share the one array, which keeps the previous call's contents;
 *     each call first clears the tickets it will use (a memset node on `stream`).  Two calls
 *     whose kernels may overlap on the GPU (different streams, no ordering) race on it:
 *     serialise them.
 *   - The first call on a device may come from several host threads at once (the set-up is
 *     guarded); the GPU-side sharing rule above is what callers have to respect.
 *   - An index outside [0, t_b) or a page id outside the pool is skipped and recorded in the
 *     array's anomaly word, which prhs_noalloc_check() reports.
 * Arguments as prhs_sparse_decode_attn, with the head counts passed explicitly.
 * Errors go to prhs_last_error(NULL). */
#define PRHS_NOALLOC_MAX_UNITS 1024
#define PRHS_NOALLOC_MAX_SPLITS 8
prhs_status prhs_sparse_decode_attn_noalloc(const void* q, const prhs_kv_view* kv, const int32_t* idx,
                                            const int32_t* count, int32_t idx_stride, int32_t batch,
                                            int32_t num_q_heads, int32_t num_kv_heads, void* out,
                                            float* out_lse, void* stream);

/* Companion of prhs_sparse_decode_attn_noalloc (the paper has no counterpart): synchronises
 * `stream`, reads the anomaly word the allocation-free calls on the current device share, and
 * clears it.  *out_flags (may be NULL) receives the PRHS_FLAG_* bits; the return value is
 * PRHS_ERR_DEVICE_FLAG if any was set, else PRHS_OK.  Allocates nothing. */
prhs_status prhs_noalloc_check(void* stream, uint32_t* out_flags);

/* Dense flash-decoding baseline (Eq. 2): attention over all i < t_b. Same outputs. */
prhs_status prhs_dense_decode_attn(prhs_ctx* ctx, const void* q, const prhs_kv_view* kv,
                                   int32_t batch, void* out, float* out_lse, void* stream);

/* One (layer, step) of the schedule (Sec. 4.4 "Parallel Acceleration": retrieval for heads
 * that need it, cached sets for the rest, attention over valid indices only).
 * Retrieves iff layer % G_L == 0 and step % s == 0; then builds the set and attends.
 * Within a step a group's first layer must be called before its other layers.
 * With the cosine gate (sim_threshold > -1) the group's first layer decides per head on the
 * device; unless the diagnostic is on, the attention of the heads that share is then launched on
 * an internal stream beside the scoring and selection of the heads that retrieve, and `stream`
 * continues when both branches have finished (event dependencies only; the step can still be
 * captured into a CUDA graph).
 *   out        device bf16 [batch][Hq][128]
 *   out_delta  device fp32 [batch][Hq] or NULL (used only with PRHS_WANT_DELTA) */
prhs_status prhs_decode_step(prhs_ctx* ctx, int32_t layer, int32_t step, const prhs_schedule* sched,
                             const void* q, const prhs_kv_view* kv, int32_t batch, void* out,
                             float* out_delta, void* stream);

/* The same step for a caller whose per-step tensors live in HOST memory (contiguous cache
 * only).  Copies q, the new token's key and value rows and seq_lens host->device, writes
 * the rows into the cache at position t_b - 1, runs prhs_decode_step, copies the output
 * device->host and synchronises the stream before returning.  When all five host buffers are
 * pinned memory that the device can address (cudaHostAlloc / cudaHostRegister under unified
 * addressing; q, k, v 16-byte aligned) the transfers are made by the kernels themselves: one
 * launch reads q, the rows and the lengths from host memory, and the attention kernel stores
 * the output into host_out.  Pageable buffers take cudaMemcpyAsync.  Results are identical.
 *   host_q [batch][Hq][128], host_new_k / host_new_v [batch][Hkv][128], host_out
 *   [batch][Hq][128]: bf16 host memory;  host_seq_lens [batch] int32 host memory.
 *   kv->k / kv->v are written (the view's const is cast away); kv->seq_lens must point to
 *   a device int32 [batch] buffer that this call overwrites. */
prhs_status prhs_decode_step_host(prhs_ctx* ctx, int32_t layer, int32_t step,
                                  const prhs_schedule* sched, const void* host_q,
                                  const void* host_new_k, const void* host_new_v,
                                  const int32_t* host_seq_lens, const prhs_kv_view* kv,
                                  int32_t batch, void* host_out, void* stream);

/* The same without the final synchronisation: everything is enqueued on `stream` and the call
 * returns.  host_q, host_new_k, host_new_v and host_seq_lens must stay unchanged, and host_out
 * is not valid, until the stream has reached the end of this call's work (the caller's own
 * cudaStreamSynchronize or event).  host_seq_lens is also read on the host, for validation,
 * during the call.  Lets a caller enqueue the next layer or step while this one runs. */
prhs_status prhs_decode_step_host_async(prhs_ctx* ctx, int32_t layer, int32_t step,
                                  const prhs_schedule* sched, const void* host_q,
                                  const void* host_new_k, const void* host_new_v,
                                  const int32_t* host_seq_lens, const prhs_kv_view* kv,
                                  int32_t batch, void* host_out, void* stream);

/* Dropped mass (Sec. 2.3): delta = 1 - sum_{i in C} A_i with A the full softmax over
 * i < t_b.  Runs a dense log-sum-exp pass and a sparse pass.  out_delta device fp32
 * [batch][Hq]. */
prhs_status prhs_delta(prhs_ctx* ctx, const void* q, const prhs_kv_view* kv, const int32_t* idx,
                       const int32_t* count, int32_t idx_stride, int32_t batch, float* out_delta,
                       void* stream);

/* Largest index-list length any call can produce: S0 + k + 2*r*m + W from prhs_config. */
int32_t prhs_index_capacity(const prhs_ctx* ctx);

/* The index set the last prhs_decode_step attended over (the step builds it inside the
 * attention kernel; this call materialises it with the stand-alone builder and copies it to
 * the host): host_idx int32 [batch][Hq][prhs_index_capacity()], host_count int32
 * [batch][Hq].  The seq_lens buffer of that step must still hold the step's lengths.
 * Synchronous; for tests and diagnostics. */
prhs_status prhs_get_index_set(prhs_ctx* ctx, int32_t batch, int32_t* host_idx,
                               int32_t* host_count, void* stream);

/* Copy the stored shared sets of `layer`'s group to the host: host_s_star (descending
 * logit) [batch][Hq][max_k], host_s_hat (ascending) [batch][Hq][max_k + 2*r*m], their
 * counts [batch][Hq] each; per head, the set it attended over in the group's latest step.
 * Any pointer may be NULL.  Synchronous. */
prhs_status prhs_get_shared_set(prhs_ctx* ctx, int32_t layer, int32_t batch, int32_t* host_s_star,
                                int32_t* host_n_star, int32_t* host_s_hat, int32_t* host_n_hat,
                                void* stream);

/* Decision of the cosine gate in the latest gated step of `layer`'s group: host_need int32
 * [batch][Hq] (1 = the head retrieved), host_ref int32 [batch][Hq] (position in the block of
 * the step it shares from, -1 = retrieved).  Either pointer may be NULL.  Synchronous. */
prhs_status prhs_get_gate(prhs_ctx* ctx, int32_t layer, int32_t batch, int32_t* host_need,
                          int32_t* host_ref, void* stream);

/* Copy the logits of the last retrieval pass to the host: fp32 [batch][Hq][ld] with
 * ld = prhs_scores_ld().  Synchronous; for tests. */
prhs_status prhs_get_scores(prhs_ctx* ctx, int32_t batch, float* host_scores, void* stream);
int32_t prhs_scores_ld(const prhs_ctx* ctx);

/* Synchronise `stream` and report: PRHS_ERR_CUDA on an asynchronous CUDA error,
 * PRHS_ERR_DEVICE_FLAG if a kernel recorded an anomaly (the flag word is then cleared;
 * *out_flags, if not NULL, receives it), else PRHS_OK. */
#define PRHS_FLAG_BAD_INDEX       1u /* an index outside [0, t_b) was skipped                */
#define PRHS_FLAG_BAD_PAGE        2u /* a page id outside [0, num_pages) was skipped          */
#define PRHS_FLAG_SELECT_FALLBACK 4u /* informational: selection took the multi-pass path     */
#define PRHS_FLAG_TIMEOUT         8u /* a bounded wait on a TMA barrier ran out; results invalid */
prhs_status prhs_check(prhs_ctx* ctx, void* stream, uint32_t* out_flags);

/* Per-kernel device timing for benchmarks (no counterpart in the paper: measurement support).
 * Between prhs_profile_begin and prhs_profile_end every kernel launch of the context is
 * bracketed by a pair of CUDA events on its stream (at most max_launches launches; later
 * ones are not recorded).  prhs_profile_end synchronises `stream` and sums the elapsed
 * milliseconds and the launch counts per kernel kind into host arrays of
 * PRHS_KERNEL_KINDS entries.  Events are created in prhs_profile_begin, not per launch. */
#define PRHS_KERNEL_KINDS 6
#define PRHS_KIND_SCORE 0        /* dense scoring (retrieval, or the delta diagnostic)  */
#define PRHS_KIND_SELECT 1       /* top-k selection + dilation                         */
#define PRHS_KIND_BUILD 2        /* index-set builder                                  */
#define PRHS_KIND_ATTN_SPARSE 3  /* gathered attention + merge                         */
#define PRHS_KIND_ATTN_DENSE 4   /* dense flash-decoding baseline                      */
#define PRHS_KIND_MISC 5         /* row append, log-sum-exp reduction                  */
prhs_status prhs_profile_begin(prhs_ctx* ctx, int32_t max_launches);
prhs_status prhs_profile_end(prhs_ctx* ctx, void* stream, float* host_ms_per_kind,
                             int64_t* host_launches_per_kind);
const char* prhs_kernel_kind_name(int32_t kind);

/* Measurement support (no counterpart in the paper): the bare row gather of
 * prhs_sparse_decode_attn, without its arithmetic.  Fetches the K row and the V row of every
 * entry of the given lists (same arguments, contiguous caches only) with the work laid out as the
 * attention kernel lays it out, and discards them.  variant: 0 = plain 16-byte loads into
 * registers, 1 = 16-byte cp.async copies into a shared-memory ring (the attention kernel's
 * mechanism), 2 = one 256-byte bulk copy per row, 3 = TMA row gather (tile::gather4, four rows per
 * instruction).  Timed with CUDA events by the caller, it gives the ceiling each mechanism sets for
 * the gathered attention on the same index pattern (python -m paper_2602_08329_b200.gather_ceiling).
 * Out-of-range entries are replaced by a valid row and flagged.  Asynchronous on `stream`. */
prhs_status prhs_gather_probe(prhs_ctx* ctx, int32_t variant, const prhs_kv_view* kv, const int32_t* idx,
                              const int32_t* count, int32_t idx_stride, int32_t batch, void* stream);

/* Number of kernels this context has launched since creation (host-side counter). */
int64_t prhs_launch_count(const prhs_ctx* ctx);

/* Diagnostic for callers that build their own lists for prhs_sparse_decode_attn: checks on the
 * device that every (b, h) list is strictly ascending (hence free of duplicates), lies inside
 * [0, t_b) and is no longer than idx_stride.  host_num_bad receives the number of offending
 * units, host_bad_units (host int32 [batch][Hq], or NULL) a 0 / 1 mark per unit.  The attention
 * kernels skip and flag out-of-range entries on their own; order and uniqueness are only
 * checked here.  Synchronises the stream. */
prhs_status prhs_validate_index_lists(prhs_ctx* ctx, const prhs_kv_view* kv, const int32_t* idx,
                                      const int32_t* count, int32_t idx_stride, int32_t batch,
                                      int32_t* host_bad_units, int32_t* host_num_bad, void* stream);

/* Checkpoint of the shared-set state (no counterpart in the paper): everything a context carries
 * from one decode step to the next -- the stored S*, S^ and their sizes per (layer group,
 * sequence, head, slot), the lengths at the last retrieval, the cosine gate's block history and
 * decisions, and where every layer group stands in its schedule -- as one flat host buffer of
 * prhs_state_bytes() bytes.  Import restores it into a context created with the SAME
 * prhs_config (PRHS_ERR_INVALID_ARG otherwise); decoding then continues as if uninterrupted,
 * bit for bit.  The KV cache itself belongs to the caller.  Both calls synchronise the stream. */
int64_t prhs_state_bytes(const prhs_ctx* ctx);
prhs_status prhs_state_export(prhs_ctx* ctx, void* host_buf, int64_t bytes, void* stream);
prhs_status prhs_state_import(prhs_ctx* ctx, const void* host_buf, int64_t bytes, void* stream);

/* Self-test of the failure path of the TMA kernels (no counterpart in the paper): launches one
 * thread that waits, with the given budget in SM cycles (1 .. 2e8, about 0.1 s), on a barrier
 * that nothing completes.  The wait must give up: *host_gave_up = 1, PRHS_FLAG_TIMEOUT is set in
 * the device flag word (the next prhs_check reports and clears it) and the context stays
 * usable.  Synchronises the stream. */
prhs_status prhs_selftest_wait(prhs_ctx* ctx, int64_t budget_cycles, int32_t* host_gave_up, void* stream);

/* Message of the last error on this context (or of the last failed prhs_create when ctx is
 * NULL).  The pointer stays valid until the next call on the context. */
const char* prhs_last_error(const prhs_ctx* ctx);

/* Library version string. */
const char* prhs_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PRHS_H_ */
