// Host side of the PrHS sparse decode-attention library: context, argument validation,
// launch configuration and the C ABI declared in include/prhs.h.
#include "../../include/prhs.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <string>
#include <vector>

#ifdef PRHS_NVTX
#include <nvtx3/nvToolsExt.h>
#endif

#include "attn.cuh"
#include "common.cuh"
#include "attn_group.cuh"
#include "score_tma.cuh"
#include "score_umma.cuh"
#include "select.cuh"
#include "gather_probe.cuh"
#include "attn_tma.cuh"
#include "attn_group_umma.cuh"

using namespace prhs;

namespace {

constexpr int kMaxSplits = 64;          // split-K partial slots per (b, h)
constexpr int kMaxSmemBytes = 227 * 1024;
constexpr int kMaxContext = 1 << 20;

std::string g_create_error;

}  // namespace

// The list of a unit is given explicitly (idx/count), by the fused builder (a SetRef: stored
// middle set plus the sink and window sizes) or, with neither, is every position (dense).

// ---- scratch of the allocation-free entry point: split-K partials, merge tickets, flag word.
// In host code the name is a stand-in, not a device address: set-up resolves it per device.
constexpr size_t kNoAllocPartialFloats =
    (size_t)PRHS_NOALLOC_MAX_UNITS * PRHS_NOALLOC_MAX_SPLITS * kPartStride;
constexpr size_t kNoAllocScratchBytes =
    kNoAllocPartialFloats * sizeof(float) + (PRHS_NOALLOC_MAX_UNITS + 64) * sizeof(unsigned int);
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

struct prhs_ctx {
  prhs_config cfg{};
  int device = 0, sm_count = 148;
  int gq = 1, num_groups = 1, max_m = 0, shat_cap = 0, idx_cap = 0, ld = 0, sort_cap = 2;
  int cand_cap = 0, two_bitmaps = 0, last_share_gq = 1;
  int max_chunks = 1, attn_ctas_per_sm = 2;
  size_t sel_smem = 0;
  // workspaces (device)
  float* scores = nullptr;
  float2* part_ml = nullptr;
  float* lse_full = nullptr;
  float* lse_c = nullptr;
  float* partials = nullptr;
  unsigned int* tickets = nullptr;
  int* idx = nullptr;
  int* count = nullptr;
  uint32_t* flags = nullptr;
  __nv_bfloat16* scratch_out = nullptr;
  // shared-set state (device), per layer group
  int *sstar_desc = nullptr, *sstar_asc = nullptr, *shat_asc = nullptr;
  int *n_star = nullptr, *n_hat = nullptr, *anchor_t = nullptr;
  // cosine gate (per layer group): block history and the decision of the latest step
  int slots = 1;                    // sets kept per (b, h) and block (= max_block_sets)
  __nv_bfloat16* qhist = nullptr;   // [G][U][slots][128] queries of the block so far
  int *set_of_pos = nullptr;        // [G][U][slots] slot each step of the block attended over
  int *nsets = nullptr;             // [G][U] sets retrieved so far in the block
  int *g_need = nullptr, *g_slot = nullptr, *g_ref = nullptr;   // [G][U] decision of the latest step
  std::vector<int> gate_step;       // host: step of each group's latest gate decision, -1 = never
  std::vector<int> anchor_step;     // host: step at which each group last retrieved, -1 = never
  // staging for the host-buffer entry point (device)
  __nv_bfloat16 *st_q = nullptr, *st_k = nullptr, *st_v = nullptr, *st_out = nullptr;
  int last_batch = 0, last_layer_group = 1, last_nchunks = 1;
  // cuTensorMapEncodeTiled, resolved at run time (no link against libcuda); nullptr = no TMA path
  void* encode_tiled = nullptr;
  // cosine-gated steps run the attention of the heads that share on this stream, beside the
  // scoring and selection of the heads that retrieve on the caller's (Fig. 6: two branches)
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // tensor maps of the gathered attention's K and V views (one row by 64 columns per box), kept
  // from call to call: encoding one costs about a microsecond of host time
  struct RowMap { const void* base; unsigned long long rows; CUtensorMap map; };
  std::vector<RowMap> row_maps;
  size_t row_map_next = 0;
  SetRef last_set{};                // what the last decode step attended over (for diagnostics)
  const int* last_seq_lens = nullptr;
  long long launches = 0;
  // optional per-launch event timing
  struct ProfRec { cudaEvent_t a, b; int kind; };
  std::vector<ProfRec> prof;
  int prof_used = 0;
  bool prof_on = false;
  std::string err;
};

namespace {

prhs_status fail(prhs_ctx* ctx, prhs_status st, const std::string& msg) {
  if (ctx) ctx->err = msg; else g_create_error = msg;
  return st;
}

#define PRHS_CUDA(ctx, expr)                                                              \
  do {                                                                                    \
    cudaError_t e_ = (expr);                                                              \
    if (e_ != cudaSuccess)                                                                \
      return fail(ctx, PRHS_ERR_CUDA, std::string(#expr) + ": " + cudaGetErrorString(e_)); \
  } while (0)

template <typename T>
cudaError_t dev_alloc(T** p, size_t n) {
  return cudaMalloc(reinterpret_cast<void**>(p), std::max<size_t>(n, 1) * sizeof(T));
}

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

size_t units_max(const prhs_ctx* c) { return (size_t)c->cfg.max_batch * c->cfg.num_q_heads; }

prhs_status check_view(prhs_ctx* ctx, const prhs_kv_view* kv, int batch, KvDev* out, int* max_t) {
  if (!kv || !kv->k || !kv->v || !kv->seq_lens) return fail(ctx, PRHS_ERR_INVALID_ARG, "kv view: NULL pointer");
  if (batch < 1) return fail(ctx, PRHS_ERR_INVALID_ARG, "batch must be >= 1");
  if (batch > ctx->cfg.max_batch) return fail(ctx, PRHS_ERR_CAPACITY, "batch exceeds max_batch");
  if ((kv->stride_outer % kHeadDim) || (kv->stride_head % kHeadDim) || ((uintptr_t)kv->k % 16) ||
      ((uintptr_t)kv->v % 16))
    return fail(ctx, PRHS_ERR_INVALID_ARG, "kv view: strides must be multiples of 128 elements and bases 16-byte aligned");
  if (kv->stride_outer <= 0 || kv->stride_head <= 0)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "kv view: strides must be positive");
  const bool paged = kv->page_table != nullptr;
  if (paged != (ctx->cfg.page_size == 16))
    return fail(ctx, PRHS_ERR_INVALID_ARG, "kv view: page table does not match the configured page_size");
  if (paged && (kv->page_table_stride < 1 || kv->num_pages < 1))
    return fail(ctx, PRHS_ERR_INVALID_ARG, "kv view: bad page table stride or pool size");
  int mt = kv->max_seq_len > 0 ? kv->max_seq_len : ctx->cfg.max_context;
  if (mt > ctx->cfg.max_context) return fail(ctx, PRHS_ERR_CAPACITY, "max_seq_len exceeds max_context");
  out->k = static_cast<const __nv_bfloat16*>(kv->k);
  out->v = static_cast<const __nv_bfloat16*>(kv->v);
  out->stride_outer = kv->stride_outer;
  out->stride_head = kv->stride_head;
  out->page_table = kv->page_table;
  out->page_table_stride = kv->page_table_stride;
  out->seq_lens = kv->seq_lens;
  out->num_pages = kv->num_pages;
  *max_t = mt;
  return PRHS_OK;
}

prhs_status check_sched(prhs_ctx* ctx, const prhs_schedule* s) {
  if (!s) return fail(ctx, PRHS_ERR_INVALID_ARG, "schedule: NULL");
  if (s->refresh_interval < 1 || s->layer_group < 1)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "schedule: refresh_interval and layer_group must be >= 1");
  if (s->layer_group < ctx->cfg.min_layer_group)
    return fail(ctx, PRHS_ERR_CAPACITY, "schedule: layer_group below min_layer_group");
  if (s->top_k < 0 || s->window < 0 || s->sinks < 0 || s->dilate_r < 0 || s->dilate_m < -1)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "schedule: negative budget");
  if (!(s->sim_threshold <= 1.f))
    return fail(ctx, PRHS_ERR_INVALID_ARG, "schedule: sim_threshold must be <= 1 (<= -1 switches the gate off)");
  if (s->psaw_layer_start < 0 ||
      (s->psaw_layer_start > 0 && !(s->psaw_phi > 0.f && s->psaw_phi < 1.f && s->psaw_alpha >= 0.f)))
    return fail(ctx, PRHS_ERR_INVALID_ARG, "schedule: sliding window needs 0 < phi < 1, alpha >= 0, l_s >= 0");
  if (s->top_k > ctx->cfg.max_k || s->window > ctx->cfg.max_window || s->sinks > ctx->cfg.max_sinks ||
      s->dilate_r > ctx->cfg.max_dilate_r || (s->dilate_m >= 0 && s->dilate_m > ctx->max_m))
    return fail(ctx, PRHS_ERR_CAPACITY, "schedule: budget exceeds the configured maximum");
  // m = floor(k / 3) by default (Sec. 5.1): the dilated set must fit what the context was sized for
  if (s->dilate_m < 0 && (s->top_k_per_seq ? ctx->cfg.max_k : s->top_k) / 3 > ctx->max_m)
    return fail(ctx, PRHS_ERR_CAPACITY, "schedule: floor(k / 3) dilated winners exceed max_dilate_m");
  if ((s->flags & PRHS_GROUP_SETS) && s->sim_threshold > -1.f)
    return fail(ctx, PRHS_ERR_UNSUPPORTED, "schedule: the cosine gate is per head, group-shared sets are per KV head");
  return PRHS_OK;
}

// Brackets one kernel launch: counts it and, in profiling mode, records an event pair.
// With -DPRHS_NVTX every launch also sits in an NVTX range named after its kind (a timeline tool
// then shows the stages of a step); off by default.
#ifdef PRHS_NVTX
static const char* const kKindNames[PRHS_KERNEL_KINDS] = {"prhs score", "prhs select", "prhs build_set",
                                                          "prhs attn_sparse", "prhs attn_dense", "prhs misc"};
#endif
struct LaunchScope {
  prhs_ctx* c;
  cudaStream_t st;
  int slot = -1;
  LaunchScope(prhs_ctx* ctx, int kind, cudaStream_t stream) : c(ctx), st(stream) {
#ifdef PRHS_NVTX
    nvtxRangePushA(kKindNames[kind]);
#endif
    c->launches++;
    if (c->prof_on && c->prof_used < (int)c->prof.size()) {
      slot = c->prof_used++;
      c->prof[slot].kind = kind;
      cudaEventRecord(c->prof[slot].a, st);
    }
  }
  ~LaunchScope() {
    if (slot >= 0) cudaEventRecord(c->prof[slot].b, st);
#ifdef PRHS_NVTX
    nvtxRangePop();
#endif
  }
};

// ---- launchers -----------------------------------------------------------------------
// Split count for the gathered attention: minimise (waves of CTAs) x (rows per CTA plus a
// fixed per-CTA cost), so that the grid fills an integer number of waves of resident CTAs.
int pick_splits(const prhs_ctx* c, int units, int max_count) {
  const int slots = c->sm_count * c->attn_ctas_per_sm;
  const int overhead_rows = 96;     // prologue + combine + partial write, in row equivalents
  int best = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= kMaxSplits; ++s) {
    const int rows = (max_count + s - 1) / s;
    if (s > 1 && rows < 64) break;
    const long long ctas = (long long)units * s;
    const double waves = (double)((ctas + slots - 1) / slots);
    const double cost = waves * (rows + overhead_rows);
    if (cost < best_cost * 0.999) { best_cost = cost; best = s; }
  }
  return best;
}

// Split count for the scoring kernels: a thousand key rows (256 KB) per CTA for a contiguous
// cache, 4096 for a paged one (whose producer pays a page-table look-up per 16 rows), and so
// several waves of CTAs per launch.  Short CTAs finish at different times, so the SMs never run
// dry together: a grid of one wave of long CTAs measured 3 to 5 % slower (the 32K-context layer
// at batch 8: 327 us against 312 us; the ragged paged batch of 64: 747 us against 711 us).  A
// small batch gets at least two CTAs per resident slot, but no CTA fewer than 256 rows.  Contexts
// of a few thousand keys are bound by latency, not by the stream: they keep the single wave.
int score_splits(const prhs_ctx* c, int units, int max_t, bool paged, bool gated) {
  if (max_t <= 8192) return pick_splits(c, units, max_t);      // short contexts are bound by latency: one wave
  const int slots = c->sm_count * 2;
  // a cosine-gated step launches the CTAs of every unit and those of the units that share return at
  // once: four times fewer CTAs there (7 us of empty CTAs per step at 8448, 2 us at 2304)
  const int rows = (paged || gated) ? 4096 : 1024;
  int s = (max_t + rows - 1) / rows;
  const int fill = (2 * slots + units - 1) / std::max(units, 1);
  s = std::max(s, std::min(fill, max_t / 256));
  return std::max(1, std::min(s, kMaxSplits));
}

// `sched` != nullptr: a retrieval pass (the fp32 logits are written for the selection kernel);
// nullptr: only the per-split log-sum-exp partials (the delta diagnostic).
prhs_status launch_score(prhs_ctx* c, const void* q, const KvDev& kv, int batch, int max_t,
                         const prhs_schedule* sched, const int* need, cudaStream_t st, int* nchunks_out) {
  const int write_scores = sched != nullptr;
  ScoreParams sp;
  sp.q = static_cast<const __nv_bfloat16*>(q);
  sp.kv = kv;
  sp.scores = write_scores ? c->scores : nullptr;
  sp.ld = c->ld;
  sp.part_ml = c->part_ml;
  sp.splits = score_splits(c, batch * c->cfg.num_kv_heads, max_t, kv.page_table != nullptr, need != nullptr);
  sp.num_q_heads = c->cfg.num_q_heads;
  sp.group_size = c->gq;
  sp.need = need;
  sp.group_max = (sched && (sched->flags & PRHS_GROUP_SETS) && c->gq > 1) ? 1 : 0;
  // A cosine-gated step launches the grid for every unit and the CTAs of the units that share return at
  // once.  CTAs of a kernel that uses tensor memory are several times slower to launch and retire even
  // then (8448 empty CTAs: 28 us against 7 us for the mma.sync kernel), so gated steps score with the
  // mma.sync kernel.
  const bool umma = !(c->cfg.flags & (PRHS_CFG_MMA_SYNC_SCORE | PRHS_CFG_NO_TMA)) && need == nullptr;
  const int tile_rows = umma ? kSUTileRows : kSTStageRows;
  sp.chunk_rows = (((max_t + sp.splits - 1) / sp.splits) + tile_rows - 1) & ~(tile_rows - 1);
  sp.flags = c->flags;
  bool tma_done = false;
  if (c->encode_tiled && !(c->cfg.flags & PRHS_CFG_NO_TMA)) {
    // K as a 2-D tensor [rows][128] bf16.  Contiguous cache: rows past the last sequence's max
    // length are out of bounds for the copy engine (zero fill), rows in between belong to the
    // cache; a copy brings the rows of one tile (128 for the tcgen05 kernel, 64 for the mma.sync one).
    // Paged cache: the rows of the page pool; a copy brings the 16 rows of one page.
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    const bool paged = kv.page_table != nullptr;
    const unsigned long long outer_rows = (unsigned long long)(kv.stride_outer >> 7);
    const unsigned long long head_rows = (unsigned long long)(kv.stride_head >> 7);
    const unsigned long long rows_total =
        (unsigned long long)((paged ? kv.num_pages : batch) - 1) * outer_rows +
        (unsigned long long)(c->cfg.num_kv_heads - 1) * head_rows + (unsigned long long)(paged ? 16 : max_t);
    if (rows_total < (1ull << 31)) {
      alignas(64) CUtensorMap tm;
      const cuuint64_t gdim[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows_total};
      const cuuint64_t gstr[1] = {(cuuint64_t)kRowBytes};
      const cuuint32_t box[2] = {64u, paged ? 16u : (cuuint32_t)tile_rows};
      const cuuint32_t estr[2] = {1u, 1u};
      const CUresult cr = reinterpret_cast<EncodeFn>(c->encode_tiled)(
          &tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(kv.k), gdim, gstr, box, estr,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (cr == CUDA_SUCCESS) {
        LaunchScope ls(c, PRHS_KIND_SCORE, st);
        const dim3 grid(sp.splits, c->cfg.num_kv_heads, batch);
        if (umma && paged) score_umma_kernel<true><<<grid, kSUThreads, kSUSmemBytes, st>>>(tm, sp);
        else if (umma) score_umma_kernel<false><<<grid, kSUThreads, kSUSmemBytes, st>>>(tm, sp);
        else if (paged) score_tma_kernel<true><<<grid, kSTThreads, kSTSmemBytes, st>>>(tm, sp);
        else score_tma_kernel<false><<<grid, kSTThreads, kSTSmemBytes, st>>>(tm, sp);
        tma_done = true;
      }
    }
  }
  if (!tma_done) {
    LaunchScope ls(c, PRHS_KIND_SCORE, st);
    score_ring_kernel<<<dim3(sp.splits, c->cfg.num_kv_heads, batch), kTThreads, kSRSmemBytes, st>>>(sp);
  }
  const int nchunks = sp.splits;
  c->last_nchunks = nchunks;
  *nchunks_out = nchunks;
  PRHS_CUDA(c, cudaGetLastError());
  return PRHS_OK;
}

// Tensor map of a K or V array viewed as [rows][128] bf16 with a box of ONE row by 64 columns and
// the 128-byte swizzle: what a tile::gather4 copy of the gathered attention names rows in.
// false if the driver cannot encode it.
bool row_gather_map(prhs_ctx* c, const void* base, unsigned long long rows, CUtensorMap* out) {
  for (const auto& m : c->row_maps)
    if (m.base == base && m.rows == rows) { *out = m.map; return true; }
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                               const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                               CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  prhs_ctx::RowMap rm;
  rm.base = base;
  rm.rows = rows;
  const cuuint64_t gdim[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
  const cuuint64_t gstr[1] = {(cuuint64_t)kRowBytes};
  const cuuint32_t box[2] = {64u, 1u};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUresult cr = reinterpret_cast<EncodeFn>(c->encode_tiled)(
      &rm.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstr, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return false;
  *out = rm.map;
  if (c->row_maps.size() < 32) {
    c->row_maps.push_back(rm);
  } else {
    c->row_maps[c->row_map_next] = rm;
    c->row_map_next = (c->row_map_next + 1) % c->row_maps.size();
  }
  return true;
}

prhs_status launch_attn(prhs_ctx* c, const void* q, const KvDev& kv, const int* idx, const int* count,
                        int idx_stride, const SetRef& fs, int max_count, int batch, void* out,
                        float* out_lse, const float* lse_full, float* out_delta, cudaStream_t st, int max_rows,
                        const int* need = nullptr, int need_mode = 0) {
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.kv = kv;
  p.idx = idx;
  p.count = count;
  p.idx_stride = idx ? idx_stride : 0x7fffffff;
  p.set = fs;
  if (idx) p.set.star = nullptr;
  p.num_q_heads = c->cfg.num_q_heads;
  p.group_size = c->gq;
  p.splits = pick_splits(c, batch * c->cfg.num_q_heads, max_count);
  p.partials = c->partials;
  p.tickets = c->tickets;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.out_lse = out_lse;
  p.lse_full = lse_full;
  p.out_delta = lse_full ? out_delta : nullptr;
  p.flags = c->flags;
  p.need = need;
  p.need_mode = need ? need_mode : 0;
  if (!idx && !fs.star) {
    // dense baseline: one CTA column per KV head, the group's heads share the K/V stream
    p.splits = pick_splits(c, batch * c->cfg.num_kv_heads, max_count);
    dim3 grid(p.splits, c->cfg.num_kv_heads, batch);
    LaunchScope ls(c, PRHS_KIND_ATTN_DENSE, st);
    dense_attn_mma_kernel<<<grid, kTThreads, kTSmemBytes, st>>>(p);
  } else if (!idx && fs.share_gq > 1) {
    // group-shared sets: one CTA column per KV head, a gathered row serves the whole group
    LaunchScope ls(c, PRHS_KIND_ATTN_SPARSE, st);
    if (c->cfg.flags & PRHS_CFG_GROUP_TCGEN05) {
      // Two shapes of CTA: 18 warps with a 205 KB ring (one per SM: the deeper pipeline), or 10 warps with
      // 109 KB (two per SM, which cover each other's set-up and merge).  The second where there are more
      // units than SMs and a launch is several waves (the ragged paged batch of 64: 128 us against 192 us
      // per sharing step; at 128 units the first: 44.5 against 56.5).  Then the split count that fills
      // whole waves of CTA slots, in tiles of 128 rows.
      const int units = batch * c->cfg.num_kv_heads;
      const bool light = units > c->sm_count;
      const int slots = c->sm_count * (light ? 2 : 1);
      int best = 1;
      double best_cost = 1e30;
      for (int s = 1; s <= kMaxSplits; ++s) {
        const int rows = (((max_count + s - 1) / s) + kGUTileRows - 1) & ~(kGUTileRows - 1);
        if (s > 1 && rows < 2 * kGUTileRows) break;
        const double waves = (double)(((long long)units * s + slots - 1) / slots);
        const double cost = waves * (rows + 2 * kGUTileRows);
        if (cost < best_cost * 0.999) { best_cost = cost; best = s; }
      }
      p.splits = best;
      dim3 grid(p.splits, c->cfg.num_kv_heads, batch);
      if (light) gather_group_attn_umma_kernel<1, 1><<<grid, GUShape<1, 1>::kThreads, GUShape<1, 1>::kSmemBytes, st>>>(p);
      else gather_group_attn_umma_kernel<2, 2><<<grid, GUShape<2, 2>::kThreads, GUShape<2, 2>::kSmemBytes, st>>>(p);
    } else {
      p.splits = pick_splits(c, batch * c->cfg.num_kv_heads, max_count);
      dim3 grid(p.splits, c->cfg.num_kv_heads, batch);
      gather_group_attn_mma_kernel<<<grid, kTThreads, kTSmemBytes, st>>>(p);
    }
  } else {
    dim3 grid(p.splits, c->cfg.num_q_heads, batch);
    // rows by 16-byte cp.async copies; by TMA row gather only where the context asks for it
    // (PRHS_CFG_TMA_GATHER: measured slower, kept for comparison)
    alignas(64) CUtensorMap tmk, tmv;
    bool have_maps = false;
    unsigned long long rows_total = 0;
    if (c->encode_tiled && (c->cfg.flags & PRHS_CFG_TMA_GATHER) && !(c->cfg.flags & PRHS_CFG_NO_TMA)) {
      const bool paged = kv.page_table != nullptr;
      rows_total = (unsigned long long)((paged ? kv.num_pages : batch) - 1) * (unsigned long long)(kv.stride_outer >> 7) +
                   (unsigned long long)(c->cfg.num_kv_heads - 1) * (unsigned long long)(kv.stride_head >> 7) +
                   (unsigned long long)(paged ? 16 : max_rows);
      if (rows_total < (1ull << 31) - 1)
        have_maps = row_gather_map(c, kv.k, rows_total, &tmk) && row_gather_map(c, kv.v, rows_total, &tmv);
    }
    LaunchScope ls(c, PRHS_KIND_ATTN_SPARSE, st);
    if (have_maps) gather_attn_tma_kernel<<<grid, kTThreads, kATSmemBytes, st>>>(tmk, tmv, p, (uint32_t)rows_total);
    else gather_attn_mma_kernel<<<grid, kTThreads, kTSmemBytes, st>>>(p);
  }
  PRHS_CUDA(c, cudaGetLastError());
  return PRHS_OK;
}

int group_of(const prhs_schedule* s, int layer) { return layer / s->layer_group; }

// Sliding-window factor c of Eq. 11 for a 0-based layer: P_l(t) = floor(c t); 0 = no window.
double psaw_factor(const prhs_ctx* c, const prhs_schedule* s, int layer) {
  const int N = c->cfg.num_layers, ls = s->psaw_layer_start, ell = layer + 1;
  if (ls <= 0 || ell < ls || N <= ls) return 0.0;
  const double expo = (double)s->psaw_alpha * (double)(ell - ls) / (double)(N - ls);
  return 1.0 - std::pow((double)s->psaw_phi, expo);
}

// Offset of a layer group's block in a state array with `per_slot` elements per (unit, slot).
size_t state_off(const prhs_ctx* c, int group, size_t per_slot) {
  return (size_t)group * units_max(c) * c->slots * per_slot;
}
// Offset of a layer group's block in a per-unit array (gate decisions, set counters).
size_t unit_off(const prhs_ctx* c, int group) { return (size_t)group * units_max(c); }

// `need` / `slot_of` (device, per unit) restrict the retrieval to the heads the cosine gate
// sent here and name the slot of the new set; nullptr = every head, slot 0.  `score_all`
// scores every head even so (the delta diagnostic wants every head's full log-sum-exp).
prhs_status do_retrieval(prhs_ctx* c, int layer, int step, const void* q, const KvDev& kv, int max_t,
                         const prhs_schedule* s, int batch, int32_t* out_idx, int32_t* out_count,
                         float* out_lse_full, const int* need, const int* slot_of, bool score_all,
                         cudaStream_t st) {
  const int g = group_of(s, layer);
  int nchunks = 1;
  prhs_status rc = launch_score(c, q, kv, batch, max_t, s, score_all ? nullptr : need, st, &nchunks);
  if (rc != PRHS_OK) return rc;
  SelectParams p;
  p.scores = c->scores;
  p.ld = c->ld;
  p.part_ml = c->part_ml;
  p.nchunks = nchunks;
  p.chunk_rows = 0;          // every split partial is written
  p.seq_lens = kv.seq_lens;
  p.k_per_seq = s->top_k_per_seq;
  p.k = s->top_k;
  p.sinks = s->sinks;
  p.window = s->window;
  p.r = s->dilate_r;
  p.m = s->dilate_m;
  p.psaw_c = psaw_factor(c, s, layer);
  p.max_k = c->cfg.max_k;
  p.shat_cap = c->shat_cap;
  p.num_q_heads = c->cfg.num_q_heads;
  p.sstar_desc = c->sstar_desc + state_off(c, g, c->cfg.max_k);
  p.sstar_asc = c->sstar_asc + state_off(c, g, c->cfg.max_k);
  p.shat_asc = c->shat_asc + state_off(c, g, c->shat_cap);
  p.n_star = c->n_star + state_off(c, g, 1);
  p.n_hat = c->n_hat + state_off(c, g, 1);
  p.need = need;
  p.slot_of = slot_of;
  p.slots = c->slots;
  p.anchor_t = c->anchor_t + (size_t)g * c->cfg.max_batch;
  p.out_idx = out_idx;
  p.out_count = out_count;
  p.lse_full = c->lse_full;
  p.out_lse_full = out_lse_full;
  p.flags = c->flags;
  p.sort_cap = c->sort_cap;
  p.cand_cap = c->cand_cap;
  p.two_bitmaps = c->two_bitmaps;
  p.unit_mul = ((s->flags & PRHS_GROUP_SETS) && c->gq > 1) ? c->gq : 1;
  {
    // One CTA of 512 threads per unit, two per SM: the kernel is a chain of short phases and wide
    // CTAs shorten it.  Where that would leave a second, partly filled wave (between two and four
    // units per SM) 256-thread CTAs, four to an SM, take all units in one wave instead (the 512
    // units of a 16 x 32-head batch: 66 us against 74 us); with at most one unit per SM the CTA
    // takes all 1024 threads (128 units of 131 K logits: 53 us against 63 us).
    const int units = batch * c->cfg.num_q_heads / p.unit_mul;
    int threads = kSelMaxThreads;
    if (units > 2 * c->sm_count && units <= 4 * c->sm_count && c->sel_smem <= 56 * 1024) threads = kSelMaxThreads / 2;
    if (units <= c->sm_count) threads = 2 * kSelMaxThreads;     // one CTA per SM at most: the widest CTA
    LaunchScope ls(c, PRHS_KIND_SELECT, st);
    select_kernel<<<units, threads, c->sel_smem, st>>>(p);
  }
  PRHS_CUDA(c, cudaGetLastError());
  if (!need) c->anchor_step[g] = step;
  c->last_layer_group = s->layer_group;
  c->last_share_gq = p.unit_mul;
  return PRHS_OK;
}

bool gated(const prhs_schedule* s) { return s->sim_threshold > -1.f; }

// The middle set (layer, step) attends over: S* for the call that retrieved it (unless
// PRHS_DILATE_ANCHOR), else the dilated S^ (Def. 3.2).  Fixed schedule: the block's first
// step on the group's first layer retrieves into slot 0.  Cosine gate: the group's first
// layer decided per head this step (need / slot), the other layers follow it.
prhs_status pick_middle(prhs_ctx* c, int layer, int step, const prhs_schedule* s, SetRef* fs) {
  const int g = group_of(s, layer);
  const int anchor = step - step % s->refresh_interval;
  const bool leader = layer % s->layer_group == 0;
  if (gated(s)) {
    if (c->gate_step[g] != step)
      return fail(c, PRHS_ERR_STATE, "no gate decision for this step: the group's first layer has not been called");
    fs->slot_of = c->g_slot + unit_off(c, g);
    fs->own_of = (leader && !(s->flags & PRHS_DILATE_ANCHOR)) ? c->g_need + unit_off(c, g) : nullptr;
    fs->own_all = 0;
  } else {
    if (c->anchor_step[g] != anchor)
      return fail(c, PRHS_ERR_STATE, "no shared set for this block: the group's first layer has not retrieved");
    fs->slot_of = nullptr;
    fs->own_of = nullptr;
    fs->own_all = (leader && step == anchor && !(s->flags & PRHS_DILATE_ANCHOR)) ? 1 : 0;
  }
  fs->star = c->sstar_asc + state_off(c, g, c->cfg.max_k);
  fs->n_star = c->n_star + state_off(c, g, 1);
  fs->hat = c->shat_asc + state_off(c, g, c->shat_cap);
  fs->n_hat = c->n_hat + state_off(c, g, 1);
  fs->star_stride = c->cfg.max_k;
  fs->hat_stride = c->shat_cap;
  fs->slots = c->slots;
  fs->share_gq = ((s->flags & PRHS_GROUP_SETS) && c->gq > 1) ? c->gq : 1;
  fs->sinks = s->sinks;
  fs->window = s->window;
  fs->psaw_c = psaw_factor(c, s, layer);
  return PRHS_OK;
}

prhs_status launch_build(prhs_ctx* c, const SetRef& fs, const int* seq_lens, int batch, int32_t* out_idx,
                         int idx_stride, int32_t* out_count, cudaStream_t st) {
  {
    LaunchScope ls(c, PRHS_KIND_BUILD, st);
    build_set_kernel<<<batch * c->cfg.num_q_heads, 128, 0, st>>>(fs, seq_lens, c->cfg.num_q_heads, out_idx,
                                                                 idx_stride, out_count);
  }
  PRHS_CUDA(c, cudaGetLastError());
  return PRHS_OK;
}

prhs_status check_layer(prhs_ctx* c, int layer, int step, const prhs_schedule* s) {
  if (layer < 0 || layer >= c->cfg.num_layers) return fail(c, PRHS_ERR_INVALID_ARG, "layer out of range");
  if (step < 0) return fail(c, PRHS_ERR_INVALID_ARG, "step must be >= 0");
  if (group_of(s, layer) >= c->num_groups) return fail(c, PRHS_ERR_CAPACITY, "layer group out of range");
  return PRHS_OK;
}

}  // namespace

// =============================================================================== C ABI
extern "C" {

const char* prhs_version(void) { return "prhs-b200 0.1"; }

const char* prhs_last_error(const prhs_ctx* ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

int64_t prhs_launch_count(const prhs_ctx* ctx) { return ctx ? ctx->launches : 0; }

prhs_status prhs_selftest_wait(prhs_ctx* ctx, int64_t budget_cycles, int32_t* host_gave_up, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (budget_cycles < 1 || budget_cycles > 200000000ll)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "selftest: budget must be in [1, 2e8] cycles");
  cudaStream_t st = as_stream(stream);
  int* d = reinterpret_cast<int*>(ctx->count);      // any device int owned by the context
  {
    LaunchScope ls(ctx, PRHS_KIND_MISC, st);
    wait_selftest_kernel<<<1, 32, 0, st>>>((long long)budget_cycles, ctx->flags, d);
  }
  PRHS_CUDA(ctx, cudaGetLastError());
  int h = -1;
  PRHS_CUDA(ctx, cudaMemcpyAsync(&h, d, sizeof(int), cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  if (host_gave_up) *host_gave_up = h;
  return PRHS_OK;
}

prhs_status prhs_validate_index_lists(prhs_ctx* ctx, const prhs_kv_view* kv, const int32_t* idx,
                                      const int32_t* count, int32_t idx_stride, int32_t batch,
                                      int32_t* host_bad_units, int32_t* host_num_bad, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!kv || !kv->seq_lens || !idx || !count || !host_num_bad) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  if (idx_stride < 1) return fail(ctx, PRHS_ERR_INVALID_ARG, "idx_stride must be >= 1");
  if (batch < 1 || batch > ctx->cfg.max_batch) return fail(ctx, PRHS_ERR_CAPACITY, "batch out of range");
  cudaStream_t st = as_stream(stream);
  const int units = batch * ctx->cfg.num_q_heads;
  int* bad = ctx->count;                       // [units] scratch of the context
  int* nbad = reinterpret_cast<int*>(ctx->tickets);   // zero between launches; restored below
  {
    LaunchScope ls(ctx, PRHS_KIND_MISC, st);
    validate_lists_kernel<<<(units + 3) / 4, 128, 0, st>>>(idx, count, idx_stride, kv->seq_lens,
                                                           ctx->cfg.num_q_heads, units, bad, nbad);
  }
  PRHS_CUDA(ctx, cudaGetLastError());
  PRHS_CUDA(ctx, cudaMemcpyAsync(host_num_bad, nbad, sizeof(int), cudaMemcpyDeviceToHost, st));
  if (host_bad_units)
    PRHS_CUDA(ctx, cudaMemcpyAsync(host_bad_units, bad, (size_t)units * sizeof(int), cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(ctx, cudaMemsetAsync(nbad, 0, sizeof(int), st));
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}

// ---- checkpoint of the shared-set state --------------------------------------------------
namespace {
constexpr uint32_t kStateMagic = 0x50724853u;   // "PrHS"
constexpr uint32_t kStateVersion = 1u;
struct StateHeader {
  uint32_t magic, version;
  prhs_config cfg;
  int32_t num_groups, slots, last_layer_group, last_share_gq;
};
struct StatePart { void* dev; size_t bytes; };
std::vector<StatePart> state_parts(prhs_ctx* c) {
  const size_t U = units_max(c), G = c->num_groups, SL = c->slots, mk = c->cfg.max_k, hc = c->shat_cap;
  return {{c->sstar_desc, G * U * SL * mk * sizeof(int)},   {c->sstar_asc, G * U * SL * mk * sizeof(int)},
          {c->shat_asc, G * U * SL * hc * sizeof(int)},     {c->n_star, G * U * SL * sizeof(int)},
          {c->n_hat, G * U * SL * sizeof(int)},             {c->anchor_t, G * c->cfg.max_batch * sizeof(int)},
          {c->qhist, G * U * SL * kHeadDim * sizeof(__nv_bfloat16)}, {c->set_of_pos, G * U * SL * sizeof(int)},
          {c->nsets, G * U * sizeof(int)},                  {c->g_need, G * U * sizeof(int)},
          {c->g_slot, G * U * sizeof(int)},                 {c->g_ref, G * U * sizeof(int)}};
}
size_t state_total(prhs_ctx* c) {
  size_t n = sizeof(StateHeader) + 2 * (size_t)c->num_groups * sizeof(int32_t);
  for (const StatePart& p : state_parts(c)) n += (p.bytes + 15) & ~(size_t)15;
  return n;
}
}  // namespace

int64_t prhs_state_bytes(const prhs_ctx* ctx) { return ctx ? (int64_t)state_total(const_cast<prhs_ctx*>(ctx)) : 0; }

prhs_status prhs_state_export(prhs_ctx* ctx, void* host_buf, int64_t bytes, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!host_buf) return fail(ctx, PRHS_ERR_INVALID_ARG, "state export: NULL buffer");
  if (bytes < (int64_t)state_total(ctx)) return fail(ctx, PRHS_ERR_CAPACITY, "state export: buffer below prhs_state_bytes()");
  cudaStream_t st = as_stream(stream);
  unsigned char* o = static_cast<unsigned char*>(host_buf);
  StateHeader h{kStateMagic, kStateVersion, ctx->cfg, ctx->num_groups, ctx->slots, ctx->last_layer_group,
                ctx->last_share_gq};
  std::memcpy(o, &h, sizeof(h));
  o += sizeof(h);
  std::memcpy(o, ctx->anchor_step.data(), ctx->num_groups * sizeof(int32_t));
  o += ctx->num_groups * sizeof(int32_t);
  std::memcpy(o, ctx->gate_step.data(), ctx->num_groups * sizeof(int32_t));
  o += ctx->num_groups * sizeof(int32_t);
  for (const StatePart& p : state_parts(ctx)) {
    PRHS_CUDA(ctx, cudaMemcpyAsync(o, p.dev, p.bytes, cudaMemcpyDeviceToHost, st));
    o += (p.bytes + 15) & ~(size_t)15;
  }
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}

prhs_status prhs_state_import(prhs_ctx* ctx, const void* host_buf, int64_t bytes, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!host_buf) return fail(ctx, PRHS_ERR_INVALID_ARG, "state import: NULL buffer");
  if (bytes < (int64_t)sizeof(StateHeader)) return fail(ctx, PRHS_ERR_INVALID_ARG, "state import: truncated buffer");
  const unsigned char* in = static_cast<const unsigned char*>(host_buf);
  StateHeader h;
  std::memcpy(&h, in, sizeof(h));
  if (h.magic != kStateMagic || h.version != kStateVersion)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "state import: not a state buffer of this library version");
  if (std::memcmp(&h.cfg, &ctx->cfg, sizeof(prhs_config)) != 0 || h.num_groups != ctx->num_groups ||
      h.slots != ctx->slots)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "state import: the buffer was exported from a different configuration");
  if (bytes < (int64_t)state_total(ctx)) return fail(ctx, PRHS_ERR_INVALID_ARG, "state import: truncated buffer");
  cudaStream_t st = as_stream(stream);
  in += sizeof(h);
  std::memcpy(ctx->anchor_step.data(), in, ctx->num_groups * sizeof(int32_t));
  in += ctx->num_groups * sizeof(int32_t);
  std::memcpy(ctx->gate_step.data(), in, ctx->num_groups * sizeof(int32_t));
  in += ctx->num_groups * sizeof(int32_t);
  for (const StatePart& p : state_parts(ctx)) {
    PRHS_CUDA(ctx, cudaMemcpyAsync(p.dev, in, p.bytes, cudaMemcpyHostToDevice, st));
    in += (p.bytes + 15) & ~(size_t)15;
  }
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  ctx->last_layer_group = h.last_layer_group;
  ctx->last_share_gq = h.last_share_gq;
  ctx->last_set = SetRef{};
  ctx->last_seq_lens = nullptr;
  ctx->last_batch = 0;
  return PRHS_OK;
}

int32_t prhs_index_capacity(const prhs_ctx* ctx) { return ctx ? ctx->idx_cap : 0; }

int32_t prhs_scores_ld(const prhs_ctx* ctx) { return ctx ? ctx->ld : 0; }

prhs_status prhs_create(const prhs_config* cfg, prhs_ctx** out) {
  if (out) *out = nullptr;
  if (!cfg || !out) return fail(nullptr, PRHS_ERR_INVALID_ARG, "prhs_create: NULL argument");
  if (cfg->head_dim != kHeadDim) return fail(nullptr, PRHS_ERR_UNSUPPORTED, "head_dim must be 128");
  if (cfg->page_size != 0 && cfg->page_size != 16)
    return fail(nullptr, PRHS_ERR_UNSUPPORTED, "page_size must be 0 or 16");
  if (cfg->num_layers < 1 || cfg->max_batch < 1 || cfg->num_q_heads < 1 || cfg->num_kv_heads < 1 ||
      cfg->max_context < 1 || cfg->max_k < 0 || cfg->max_window < 0 || cfg->max_sinks < 0 ||
      cfg->max_dilate_r < 0 || cfg->max_dilate_m < -1 || cfg->min_layer_group < 1 ||
      cfg->max_block_sets < 1 || cfg->max_block_sets > 64)
    return fail(nullptr, PRHS_ERR_INVALID_ARG, "prhs_create: non-positive size");
  if (cfg->num_q_heads % cfg->num_kv_heads) return fail(nullptr, PRHS_ERR_INVALID_ARG, "Hkv must divide Hq");
  if (cfg->num_q_heads / cfg->num_kv_heads > 16) return fail(nullptr, PRHS_ERR_UNSUPPORTED, "group size above 16");
  if (cfg->max_context > kMaxContext) return fail(nullptr, PRHS_ERR_UNSUPPORTED, "max_context above 2^20");
  if (cfg->max_k > 65536) return fail(nullptr, PRHS_ERR_UNSUPPORTED, "max_k above 65536");
  if (cfg->flags & ~(PRHS_CFG_NO_TMA | PRHS_CFG_TMA_GATHER | PRHS_CFG_MMA_SYNC_SCORE | PRHS_CFG_GROUP_TCGEN05)) return fail(nullptr, PRHS_ERR_INVALID_ARG, "prhs_create: unknown configuration flag");

  prhs_ctx* c = new (std::nothrow) prhs_ctx();
  if (!c) return fail(nullptr, PRHS_ERR_OOM, "host allocation failed");
  c->cfg = *cfg;
  c->gq = cfg->num_q_heads / cfg->num_kv_heads;
  c->num_groups = (cfg->num_layers + cfg->min_layer_group - 1) / cfg->min_layer_group;
  c->max_m = cfg->max_dilate_m < 0 ? cfg->max_k / 3 : cfg->max_dilate_m;
  c->shat_cap = cfg->max_k + 2 * cfg->max_dilate_r * c->max_m;
  c->idx_cap = cfg->max_sinks + c->shat_cap + cfg->max_window;
  c->ld = (cfg->max_context + 63) & ~63;
  c->max_chunks = kMaxSplits;
  while (c->sort_cap < cfg->max_k) c->sort_cap <<= 1;
  c->sort_cap <<= 1;   // room for a tie group that straddles the k-th place
  c->sort_cap = std::max(c->sort_cap, 64);   // the block sort works on 64-entry blocks
  c->anchor_step.assign(c->num_groups, -1);
  c->gate_step.assign(c->num_groups, -1);
  c->slots = cfg->max_block_sets;

  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device);
  if (e != cudaSuccess) {
    std::string msg = std::string("no usable CUDA device: ") + cudaGetErrorString(e);
    delete c;
    return fail(nullptr, PRHS_ERR_CUDA, msg);
  }
  // selection kernel shared memory: histograms + scalars + the candidate list (which later holds
  // the sorted entries and the merge sort's second buffer) + one or two position bitmaps
  {
    const size_t fixed = (size_t)(kHistWords + kSelMiscWords) * 4;
    const size_t bitmap_bytes = (size_t)((cfg->max_context + 31) / 32) * 4;
    auto need = [&](int cand_cap, int nbm) { return fixed + (size_t)cand_cap * 8 + nbm * bitmap_bytes; };
    c->cand_cap = std::max(4096, 2 * c->sort_cap);
    c->two_bitmaps = 1;
    if (need(c->cand_cap, 2) > (size_t)kMaxSmemBytes) c->two_bitmaps = 0;
    while (need(c->cand_cap, 1 + c->two_bitmaps) > (size_t)kMaxSmemBytes && c->cand_cap > c->sort_cap)
      c->cand_cap >>= 1;
    c->sel_smem = need(c->cand_cap, 1 + c->two_bitmaps);
  }
  if (c->sel_smem > (size_t)kMaxSmemBytes) {
    delete c;
    return fail(nullptr, PRHS_ERR_UNSUPPORTED, "max_context / max_k too large for the selection kernel");
  }
  // the opt-in limit is a property of the kernel, not of this context: always the maximum, so that
  // contexts of different sizes can live side by side
  e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_group_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_group_attn_umma_kernel<2, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, GUShape<2, 2>::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_group_attn_umma_kernel<1, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, GUShape<1, 1>::kSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(score_tma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSTSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(score_tma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSTSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(score_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSUSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(score_umma_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSUSmemBytes);
  if (e == cudaSuccess) {
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      c->encode_tiled = fn;
    else
      cudaGetLastError();      // no TMA path: the cp.async ring kernel serves every layout
  }
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(score_ring_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSRSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_attn_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kATSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_probe_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGPSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_probe_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGPSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_probe_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGPSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(gather_probe_kernel<3>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGPSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(dense_attn_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTSmemBytes);
  if (e == cudaSuccess) {
    int nb = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&nb, gather_attn_mma_kernel, kTThreads, kTSmemBytes);
    if (e == cudaSuccess && nb > 0) c->attn_ctas_per_sm = nb;
  }

  if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&c->side_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming);
  const size_t U = units_max(c), G = c->num_groups;
  if (e == cudaSuccess) e = dev_alloc(&c->scores, U * c->ld);
  if (e == cudaSuccess) e = dev_alloc(&c->part_ml, U * std::max(c->max_chunks, kMaxSplits));
  if (e == cudaSuccess) e = dev_alloc(&c->lse_full, U);
  if (e == cudaSuccess) e = dev_alloc(&c->lse_c, U);
  if (e == cudaSuccess) e = dev_alloc(&c->partials, U * kMaxSplits * kPartStride);
  if (e == cudaSuccess) e = dev_alloc(&c->tickets, U);
  if (e == cudaSuccess) e = dev_alloc(&c->idx, U * c->idx_cap);
  if (e == cudaSuccess) e = dev_alloc(&c->count, U);
  if (e == cudaSuccess) e = dev_alloc(&c->flags, 1);
  if (e == cudaSuccess) e = dev_alloc(&c->scratch_out, U * kHeadDim);
  const size_t SL = (size_t)c->slots;
  if (e == cudaSuccess) e = dev_alloc(&c->sstar_desc, G * U * SL * cfg->max_k);
  if (e == cudaSuccess) e = dev_alloc(&c->sstar_asc, G * U * SL * cfg->max_k);
  if (e == cudaSuccess) e = dev_alloc(&c->shat_asc, G * U * SL * c->shat_cap);
  if (e == cudaSuccess) e = dev_alloc(&c->n_star, G * U * SL);
  if (e == cudaSuccess) e = dev_alloc(&c->n_hat, G * U * SL);
  if (e == cudaSuccess) e = dev_alloc(&c->qhist, G * U * SL * kHeadDim);
  if (e == cudaSuccess) e = dev_alloc(&c->set_of_pos, G * U * SL);
  if (e == cudaSuccess) e = dev_alloc(&c->nsets, G * U);
  if (e == cudaSuccess) e = dev_alloc(&c->g_need, G * U);
  if (e == cudaSuccess) e = dev_alloc(&c->g_slot, G * U);
  if (e == cudaSuccess) e = dev_alloc(&c->g_ref, G * U);
  if (e == cudaSuccess) e = dev_alloc(&c->anchor_t, G * cfg->max_batch);
  if (e == cudaSuccess) e = dev_alloc(&c->st_q, U * kHeadDim);
  if (e == cudaSuccess) e = dev_alloc(&c->st_out, U * kHeadDim);
  if (e == cudaSuccess) e = dev_alloc(&c->st_k, (size_t)cfg->max_batch * cfg->num_kv_heads * kHeadDim);
  if (e == cudaSuccess) e = dev_alloc(&c->st_v, (size_t)cfg->max_batch * cfg->num_kv_heads * kHeadDim);
  if (e == cudaSuccess) e = cudaMemset(c->tickets, 0, U * sizeof(unsigned int));
  if (e == cudaSuccess) e = cudaMemset(c->flags, 0, sizeof(uint32_t));
  if (e == cudaSuccess) e = cudaMemset(c->n_star, 0, G * U * SL * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->n_hat, 0, G * U * SL * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->set_of_pos, 0, G * U * SL * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->nsets, 0, G * U * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->g_need, 0, G * U * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->g_slot, 0, G * U * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->g_ref, 0xff, G * U * sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(c->count, 0, U * sizeof(int));
  if (e != cudaSuccess) {
    std::string msg = std::string("prhs_create: ") + cudaGetErrorString(e);
    const bool oom = (e == cudaErrorMemoryAllocation);
    cudaGetLastError();
    prhs_destroy(c);
    return fail(nullptr, oom ? PRHS_ERR_OOM : PRHS_ERR_CUDA, msg);
  }
  *out = c;
  return PRHS_OK;
}

prhs_status prhs_destroy(prhs_ctx* c) {
  if (!c) return PRHS_OK;
  void* ptrs[] = {c->scores, c->part_ml, c->lse_full, c->lse_c, c->partials, c->tickets, c->idx,
                  c->count, c->flags, c->scratch_out, c->sstar_desc, c->sstar_asc, c->shat_asc,
                  c->n_star, c->n_hat, c->anchor_t, c->qhist, c->set_of_pos, c->nsets, c->g_need,
                  c->g_slot, c->g_ref, c->st_q, c->st_out, c->st_k, c->st_v};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  for (auto& r : c->prof) {
    cudaEventDestroy(r.a);
    cudaEventDestroy(r.b);
  }
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  if (c->side_stream) cudaStreamDestroy(c->side_stream);
  delete c;
  return PRHS_OK;
}

prhs_status prhs_score_topk(prhs_ctx* ctx, int32_t layer, int32_t step, const void* q,
                            const prhs_kv_view* kv, const prhs_schedule* sched, int32_t batch,
                            int32_t* out_idx, int32_t* out_count, float* out_lse_full, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!q) return fail(ctx, PRHS_ERR_INVALID_ARG, "q is NULL");
  prhs_status rc = check_sched(ctx, sched);
  if (rc != PRHS_OK) return rc;
  rc = check_layer(ctx, layer, step, sched);
  if (rc != PRHS_OK) return rc;
  if (layer % sched->layer_group) return fail(ctx, PRHS_ERR_INVALID_ARG, "retrieval runs on the first layer of a group");
  KvDev dv;
  int max_t;
  rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  return do_retrieval(ctx, layer, step, q, dv, max_t, sched, batch, out_idx, out_count, out_lse_full,
                      nullptr, nullptr, false, as_stream(stream));
}

prhs_status prhs_build_index_set(prhs_ctx* ctx, int32_t layer, int32_t step, const prhs_schedule* sched,
                                 const prhs_kv_view* kv, int32_t batch, int32_t* out_idx,
                                 int32_t idx_stride, int32_t* out_count, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!out_idx || !out_count) return fail(ctx, PRHS_ERR_INVALID_ARG, "output pointer is NULL");
  prhs_status rc = check_sched(ctx, sched);
  if (rc != PRHS_OK) return rc;
  rc = check_layer(ctx, layer, step, sched);
  if (rc != PRHS_OK) return rc;
  if (idx_stride < ctx->idx_cap) return fail(ctx, PRHS_ERR_CAPACITY, "idx_stride below prhs_index_capacity()");
  KvDev dv;
  int max_t;
  rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  SetRef fs{};
  rc = pick_middle(ctx, layer, step, sched, &fs);
  if (rc != PRHS_OK) return rc;
  return launch_build(ctx, fs, dv.seq_lens, batch, out_idx, idx_stride, out_count, as_stream(stream));
}

prhs_status prhs_sparse_decode_attn(prhs_ctx* ctx, const void* q, const prhs_kv_view* kv,
                                    const int32_t* idx, const int32_t* count, int32_t idx_stride,
                                    int32_t batch, void* out, float* out_lse, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!q || !idx || !count || !out) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  if (idx_stride < 1) return fail(ctx, PRHS_ERR_INVALID_ARG, "idx_stride must be >= 1");
  KvDev dv;
  int max_t;
  prhs_status rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  return launch_attn(ctx, q, dv, idx, count, idx_stride, SetRef{}, idx_stride, batch, out, out_lse,
                     nullptr, nullptr, as_stream(stream), max_t);
}

namespace {
// Per-device set-up state of the allocation-free entry points (no allocation): the scratch
// array's device address, SM count, resident CTAs per SM.  Guarded by a mutex so that two host
// threads may make the first call on a device at the same time.
struct NoAllocDev { unsigned char* scratch = nullptr; int sm_count = 0; int ctas_per_sm = 0; };
NoAllocDev g_noalloc_dev[64];
std::mutex g_noalloc_mutex;

// Resolves the state of the current device, doing the one-time set-up on the first call there.
prhs_status noalloc_device(NoAllocDev** out) {
  int dev = -1;
  PRHS_CUDA(nullptr, cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return fail(nullptr, PRHS_ERR_UNSUPPORTED, "noalloc: device ordinal above 63");
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  NoAllocDev& ds = g_noalloc_dev[dev];
  if (!ds.scratch) {
    // first call on this device, with this device current: in host code the array's name is a
    // stand-in, its device address has to be asked for
    unsigned char* ptr = nullptr;
    PRHS_CUDA(nullptr, cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch));
    PRHS_CUDA(nullptr, cudaFuncSetAttribute(gather_attn_mma_kernel,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kTSmemBytes));
    PRHS_CUDA(nullptr, cudaDeviceGetAttribute(&ds.sm_count, cudaDevAttrMultiProcessorCount, dev));
    PRHS_CUDA(nullptr, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&ds.ctas_per_sm, gather_attn_mma_kernel,
                                                                     kTThreads, kTSmemBytes));
    if (ds.ctas_per_sm < 1) ds.ctas_per_sm = 1;
    ds.scratch = ptr;
  }
  *out = &ds;
  return PRHS_OK;
}
inline unsigned int* noalloc_tickets(const NoAllocDev& ds) {
  return reinterpret_cast<unsigned int*>(ds.scratch + kNoAllocPartialFloats * sizeof(float));
}
}  // namespace

prhs_status prhs_sparse_decode_attn_noalloc(const void* q, const prhs_kv_view* kv, const int32_t* idx,
                                            const int32_t* count, int32_t idx_stride, int32_t batch,
                                            int32_t num_q_heads, int32_t num_kv_heads, void* out,
                                            float* out_lse, void* stream) {
  if (!q || !kv || !kv->k || !kv->v || !kv->seq_lens || !idx || !count || !out)
    return fail(nullptr, PRHS_ERR_INVALID_ARG, "noalloc: NULL pointer");
  if (batch < 1 || num_q_heads < 1 || num_kv_heads < 1 || num_q_heads % num_kv_heads || idx_stride < 1)
    return fail(nullptr, PRHS_ERR_INVALID_ARG, "noalloc: bad shape");
  if (num_q_heads / num_kv_heads > 16) return fail(nullptr, PRHS_ERR_UNSUPPORTED, "noalloc: group size above 16");
  if ((long long)batch * num_q_heads > PRHS_NOALLOC_MAX_UNITS)
    return fail(nullptr, PRHS_ERR_CAPACITY, "noalloc: batch * num_q_heads exceeds PRHS_NOALLOC_MAX_UNITS");
  if ((kv->stride_outer % kHeadDim) || (kv->stride_head % kHeadDim) || kv->stride_outer <= 0 ||
      kv->stride_head <= 0 || ((uintptr_t)kv->k % 16) || ((uintptr_t)kv->v % 16))
    return fail(nullptr, PRHS_ERR_INVALID_ARG, "noalloc: strides must be positive multiples of 128 elements, bases 16-byte aligned");
  if (kv->page_table && (kv->page_table_stride < 1 || kv->num_pages < 1))
    return fail(nullptr, PRHS_ERR_INVALID_ARG, "noalloc: bad page table stride or pool size");
  NoAllocDev* dsp = nullptr;
  prhs_status rc = noalloc_device(&dsp);
  if (rc != PRHS_OK) return rc;
  const NoAllocDev& ds = *dsp;
  cudaStream_t st = as_stream(stream);
  const int units = batch * num_q_heads;
  // same split rule as the context-based call, capped by the static capacity
  const int slots = ds.sm_count * ds.ctas_per_sm;
  int splits = 1;
  double best_cost = 1e30;
  for (int s = 1; s <= PRHS_NOALLOC_MAX_SPLITS; ++s) {
    const int rows = (idx_stride + s - 1) / s;
    if (s > 1 && rows < 64) break;
    const double waves = (double)(((long long)units * s + slots - 1) / slots);
    const double cost = waves * (rows + 96);
    if (cost < best_cost * 0.999) { best_cost = cost; splits = s; }
  }
  float* partials = reinterpret_cast<float*>(ds.scratch);
  unsigned int* tickets = noalloc_tickets(ds);
  uint32_t* flag_word = tickets + PRHS_NOALLOC_MAX_UNITS;
  // the array keeps the last call's contents: tickets must start at zero
  PRHS_CUDA(nullptr, cudaMemsetAsync(tickets, 0, (size_t)units * sizeof(unsigned int), st));
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.kv.k = static_cast<const __nv_bfloat16*>(kv->k);
  p.kv.v = static_cast<const __nv_bfloat16*>(kv->v);
  p.kv.stride_outer = kv->stride_outer;
  p.kv.stride_head = kv->stride_head;
  p.kv.page_table = kv->page_table;
  p.kv.page_table_stride = kv->page_table_stride;
  p.kv.seq_lens = kv->seq_lens;
  p.kv.num_pages = kv->num_pages;
  p.idx = idx;
  p.count = count;
  p.idx_stride = idx_stride;
  p.set = SetRef{};
  p.num_q_heads = num_q_heads;
  p.group_size = num_q_heads / num_kv_heads;
  p.splits = splits;
  p.partials = partials;
  p.tickets = tickets;
  p.out = static_cast<__nv_bfloat16*>(out);
  p.out_lse = out_lse;
  p.lse_full = nullptr;
  p.out_delta = nullptr;
  p.flags = flag_word;
  p.need = nullptr;
  p.need_mode = 0;
  gather_attn_mma_kernel<<<dim3(splits, num_q_heads, batch), kTThreads, kTSmemBytes, st>>>(p);
  PRHS_CUDA(nullptr, cudaGetLastError());
  return PRHS_OK;
}

prhs_status prhs_noalloc_check(void* stream, uint32_t* out_flags) {
  NoAllocDev* dsp = nullptr;
  prhs_status rc = noalloc_device(&dsp);
  if (rc != PRHS_OK) return rc;
  cudaStream_t st = as_stream(stream);
  uint32_t* flag_word = noalloc_tickets(*dsp) + PRHS_NOALLOC_MAX_UNITS;
  uint32_t f = 0;
  PRHS_CUDA(nullptr, cudaMemcpyAsync(&f, flag_word, sizeof(f), cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(nullptr, cudaStreamSynchronize(st));
  if (out_flags) *out_flags = f;
  if (f) {
    PRHS_CUDA(nullptr, cudaMemsetAsync(flag_word, 0, sizeof(uint32_t), st));
    PRHS_CUDA(nullptr, cudaStreamSynchronize(st));
    char buf[96];
    snprintf(buf, sizeof buf, "noalloc: device flag word 0x%x", f);
    return fail(nullptr, PRHS_ERR_DEVICE_FLAG, buf);
  }
  return PRHS_OK;
}

prhs_status prhs_gather_probe(prhs_ctx* ctx, int32_t variant, const prhs_kv_view* kv, const int32_t* idx,
                              const int32_t* count, int32_t idx_stride, int32_t batch, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!idx || !count) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  if (idx_stride < 1) return fail(ctx, PRHS_ERR_INVALID_ARG, "idx_stride must be >= 1");
  if (variant < 0 || variant > 3) return fail(ctx, PRHS_ERR_INVALID_ARG, "gather probe: variant must be 0..3");
  KvDev dv;
  int max_t;
  prhs_status rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  if (dv.page_table) return fail(ctx, PRHS_ERR_UNSUPPORTED, "gather probe: contiguous caches only");
  cudaStream_t st = as_stream(stream);
  GatherProbeParams p;
  p.kv = dv;
  p.idx = idx;
  p.count = count;
  p.idx_stride = idx_stride;
  p.num_q_heads = ctx->cfg.num_q_heads;
  p.group_size = ctx->gq;
  p.splits = pick_splits(ctx, batch * ctx->cfg.num_q_heads, idx_stride);
  p.flags = ctx->flags;
  p.sink = reinterpret_cast<unsigned int*>(ctx->lse_c);      // any word of the context; never written
  alignas(64) CUtensorMap tmk, tmv;
  std::memset(&tmk, 0, sizeof tmk);
  std::memset(&tmv, 0, sizeof tmv);
  if (variant == 3) {
    // K and V as [rows][128] bf16, a box of ONE row: a gather4 copy names four rows and brings 4 boxes
    if (!ctx->encode_tiled) return fail(ctx, PRHS_ERR_UNSUPPORTED, "gather probe: the driver offers no tensor-map encoder");
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                 const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                 CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    const unsigned long long rows_total = (unsigned long long)(batch - 1) * (unsigned long long)(dv.stride_outer >> 7) +
                                          (unsigned long long)(ctx->cfg.num_kv_heads - 1) * (unsigned long long)(dv.stride_head >> 7) +
                                          (unsigned long long)max_t;
    if (rows_total >= (1ull << 31)) return fail(ctx, PRHS_ERR_UNSUPPORTED, "gather probe: more than 2^31 rows");
    const cuuint64_t gdim[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows_total};
    const cuuint64_t gstr[1] = {(cuuint64_t)kRowBytes};
    const cuuint32_t box[2] = {(cuuint32_t)kHeadDim, 1u};
    const cuuint32_t estr[2] = {1u, 1u};
    for (int i = 0; i < 2; ++i) {
      const CUresult cr = reinterpret_cast<EncodeFn>(ctx->encode_tiled)(
          i == 0 ? &tmk : &tmv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(i == 0 ? dv.k : dv.v),
          gdim, gstr, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
          CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
      if (cr != CUDA_SUCCESS) return fail(ctx, PRHS_ERR_CUDA, "gather probe: cuTensorMapEncodeTiled failed");
    }
  }
  const dim3 grid(p.splits, ctx->cfg.num_q_heads, batch);
  {
    LaunchScope ls(ctx, PRHS_KIND_MISC, st);
    switch (variant) {
      case 0: gather_probe_kernel<0><<<grid, kTThreads, kGPSmemBytes, st>>>(tmk, tmv, p); break;
      case 1: gather_probe_kernel<1><<<grid, kTThreads, kGPSmemBytes, st>>>(tmk, tmv, p); break;
      case 2: gather_probe_kernel<2><<<grid, kTThreads, kGPSmemBytes, st>>>(tmk, tmv, p); break;
      default: gather_probe_kernel<3><<<grid, kTThreads, kGPSmemBytes, st>>>(tmk, tmv, p); break;
    }
  }
  PRHS_CUDA(ctx, cudaGetLastError());
  return PRHS_OK;
}

prhs_status prhs_dense_decode_attn(prhs_ctx* ctx, const void* q, const prhs_kv_view* kv, int32_t batch,
                                   void* out, float* out_lse, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!q || !out) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  KvDev dv;
  int max_t;
  prhs_status rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  return launch_attn(ctx, q, dv, nullptr, nullptr, 0, SetRef{}, max_t, batch, out, out_lse, nullptr,
                     nullptr, as_stream(stream), max_t);
}

prhs_status prhs_decode_step(prhs_ctx* ctx, int32_t layer, int32_t step, const prhs_schedule* sched,
                             const void* q, const prhs_kv_view* kv, int32_t batch, void* out,
                             float* out_delta, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!q || !out) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  prhs_status rc = check_sched(ctx, sched);
  if (rc != PRHS_OK) return rc;
  rc = check_layer(ctx, layer, step, sched);
  if (rc != PRHS_OK) return rc;
  KvDev dv;
  int max_t;
  rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  cudaStream_t st = as_stream(stream);
  const bool want_delta = (sched->flags & PRHS_WANT_DELTA) && out_delta;
  const bool leader = layer % sched->layer_group == 0;
  const int g = group_of(sched, layer);
  bool scored = false;                       // lse_full of every head is fresh
  if (gated(sched)) {
    // cosine gate (Eq. 9): the group's first layer decides per head, on the device, whether it
    // shares or retrieves; scoring and selection are launched every step and skip the heads
    // (and KV heads) that share
    if (sched->refresh_interval > ctx->slots)
      return fail(ctx, PRHS_ERR_CAPACITY, "cosine gate needs max_block_sets >= refresh_interval");
    if (leader) {
      const int units = batch * ctx->cfg.num_q_heads;
      const int pos = step % sched->refresh_interval;
      if (pos > 0 && ctx->gate_step[g] != step - 1)
        return fail(ctx, PRHS_ERR_STATE, "cosine gate: the previous step of this block was not run");
      int* need = ctx->g_need + unit_off(ctx, g);
      int* slot = ctx->g_slot + unit_off(ctx, g);
      {
        LaunchScope ls(ctx, PRHS_KIND_MISC, st);
        gate_kernel<<<(units + 3) / 4, 128, 0, st>>>(
            static_cast<const __nv_bfloat16*>(q), units, pos, sched->sim_threshold, ctx->slots,
            ctx->qhist + state_off(ctx, g, kHeadDim), ctx->set_of_pos + state_off(ctx, g, 1),
            ctx->nsets + unit_off(ctx, g), need, slot, ctx->g_ref + unit_off(ctx, g));
      }
      PRHS_CUDA(ctx, cudaGetLastError());
      ctx->gate_step[g] = step;
      if (!want_delta) {
        // The two branches of Fig. 6.  The heads that share attend over their cached sets on a
        // second stream while the heads that retrieve are scored and selected on the caller's;
        // the attention of the retrieving heads follows the selection, and the caller's stream
        // continues when both branches are done (events; nothing waits on the device).  The
        // diagnostic (delta) needs every head's full log-sum-exp first: no second branch then.
        SetRef fs{};
        rc = pick_middle(ctx, layer, step, sched, &fs);
        if (rc != PRHS_OK) return rc;
        ctx->last_set = fs;
        ctx->last_seq_lens = dv.seq_lens;
        ctx->last_batch = batch;
        PRHS_CUDA(ctx, cudaEventRecord(ctx->ev_fork, st));
        PRHS_CUDA(ctx, cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0));
        rc = launch_attn(ctx, q, dv, nullptr, nullptr, 0, fs, ctx->idx_cap, batch, out, ctx->lse_c, nullptr, nullptr,
                         ctx->side_stream, max_t, need, 1);
        if (rc == PRHS_OK) {
          PRHS_CUDA(ctx, cudaEventRecord(ctx->ev_join, ctx->side_stream));
          rc = do_retrieval(ctx, layer, step, q, dv, max_t, sched, batch, nullptr, nullptr, nullptr, need, slot,
                            false, st);
        }
        if (rc == PRHS_OK)
          rc = launch_attn(ctx, q, dv, nullptr, nullptr, 0, fs, ctx->idx_cap, batch, out, ctx->lse_c, nullptr, nullptr,
                           st, max_t, need, 2);
        // the side branch joins even after a failed launch, so that a capture in progress stays well formed
        const cudaError_t je = cudaStreamWaitEvent(st, ctx->ev_join, 0);
        if (rc == PRHS_OK && je != cudaSuccess) return fail(ctx, PRHS_ERR_CUDA, cudaGetErrorString(je));
        return rc;
      }
      rc = do_retrieval(ctx, layer, step, q, dv, max_t, sched, batch, nullptr, nullptr, nullptr, need, slot,
                        want_delta, st);
      if (rc != PRHS_OK) return rc;
      if (want_delta) {        // every head was scored; heads that share still need their lse_full
        const int n = batch * ctx->cfg.num_q_heads;
        LaunchScope ls(ctx, PRHS_KIND_MISC, st);
        lse_reduce_kernel<<<(n + 127) / 128, 128, 0, st>>>(ctx->part_ml, ctx->last_nchunks, 0, dv.seq_lens,
                                                           ctx->cfg.num_q_heads, ctx->lse_full, n);
        scored = true;
      }
    }
  } else if (leader && step % sched->refresh_interval == 0) {
    rc = do_retrieval(ctx, layer, step, q, dv, max_t, sched, batch, nullptr, nullptr, nullptr, nullptr, nullptr,
                      false, st);
    if (rc != PRHS_OK) return rc;
    scored = true;
  }
  if (want_delta && !scored) {
    int nchunks = 1;
    rc = launch_score(ctx, q, dv, batch, max_t, nullptr, nullptr, st, &nchunks);
    if (rc != PRHS_OK) return rc;
    const int n = batch * ctx->cfg.num_q_heads;
    {
      LaunchScope ls(ctx, PRHS_KIND_MISC, st);
      lse_reduce_kernel<<<(n + 127) / 128, 128, 0, st>>>(ctx->part_ml, nchunks, 0, dv.seq_lens,
                                                         ctx->cfg.num_q_heads, ctx->lse_full, n);
    }
    PRHS_CUDA(ctx, cudaGetLastError());
  }
  // the index set is built inside the attention kernel from the stored middle set
  SetRef fs{};
  rc = pick_middle(ctx, layer, step, sched, &fs);
  if (rc != PRHS_OK) return rc;
  ctx->last_set = fs;
  ctx->last_seq_lens = dv.seq_lens;
  ctx->last_batch = batch;
  return launch_attn(ctx, q, dv, nullptr, nullptr, 0, fs, ctx->idx_cap, batch, out, ctx->lse_c,
                     want_delta ? ctx->lse_full : nullptr, want_delta ? out_delta : nullptr, st, max_t);
}

namespace {
prhs_status decode_step_host_impl(prhs_ctx* ctx, int32_t layer, int32_t step, const prhs_schedule* sched,
                                  const void* host_q, const void* host_new_k, const void* host_new_v,
                                  const int32_t* host_seq_lens, const prhs_kv_view* kv, int32_t batch,
                                  void* host_out, void* stream, bool sync) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!host_q || !host_new_k || !host_new_v || !host_seq_lens || !host_out || !kv)
    return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  if (kv->page_table) return fail(ctx, PRHS_ERR_UNSUPPORTED, "host entry point needs a contiguous cache");
  // everything prhs_decode_step would reject is rejected here, before the cache is written
  prhs_status vrc = check_sched(ctx, sched);
  if (vrc != PRHS_OK) return vrc;
  vrc = check_layer(ctx, layer, step, sched);
  if (vrc != PRHS_OK) return vrc;
  {
    KvDev unused;
    int cap = 0;
    vrc = check_view(ctx, kv, batch, &unused, &cap);
    if (vrc != PRHS_OK) return vrc;
    // the new row lands at position t_b - 1 of the (b, kvh) slice: it must lie inside the capacity
    // the view declares and inside the slice itself (a slice ends where the next head or sequence begins)
    const long long slice_rows = std::min(kv->stride_head, kv->stride_outer) / kHeadDim;
    for (int b = 0; b < batch; ++b) {
      if (host_seq_lens[b] < 1) return fail(ctx, PRHS_ERR_INVALID_ARG, "seq_lens entry below 1");
      if (host_seq_lens[b] > cap || host_seq_lens[b] > slice_rows)
        return fail(ctx, PRHS_ERR_CAPACITY, "seq_lens entry exceeds the cache capacity (max_seq_len, strides)");
    }
  }
  cudaStream_t st = as_stream(stream);
  const size_t qb = (size_t)batch * ctx->cfg.num_q_heads * kRowBytes;
  const size_t kb = (size_t)batch * ctx->cfg.num_kv_heads * kRowBytes;
  // Pinned host buffers that the device can address (what cudaHostAlloc / cudaHostRegister give
  // under unified addressing) are read and written by the kernels themselves: one ingest launch
  // instead of four copies and an append, and the attention kernel stores the result where the
  // caller wants it.  Anything else (pageable memory) goes through cudaMemcpyAsync.
  auto mapped = [](const void* p) -> void* {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
  };
  void* dq = mapped(host_q);
  void* dk = dq ? mapped(host_new_k) : nullptr;
  void* dv = dk ? mapped(host_new_v) : nullptr;
  void* dl = dv ? mapped(host_seq_lens) : nullptr;
  void* dout = dl ? mapped(host_out) : nullptr;
  const bool aligned = (((uintptr_t)dq | (uintptr_t)dk | (uintptr_t)dv) & 15u) == 0 && ((uintptr_t)dl & 3u) == 0 &&
                       ((uintptr_t)dout & 1u) == 0;
  if (dout && aligned) {
    {
      LaunchScope ls(ctx, PRHS_KIND_MISC, st);
      ingest_kernel<<<dim3(batch, kIngestSplit), 256, 0, st>>>(
          static_cast<const uint4*>(dq), static_cast<const uint4*>(dk), static_cast<const uint4*>(dv),
          static_cast<const int*>(dl), reinterpret_cast<uint4*>(ctx->st_q),
          static_cast<__nv_bfloat16*>(const_cast<void*>(kv->k)), static_cast<__nv_bfloat16*>(const_cast<void*>(kv->v)),
          kv->stride_outer, kv->stride_head, const_cast<int32_t*>(kv->seq_lens), ctx->cfg.num_q_heads,
          ctx->cfg.num_kv_heads);
    }
    PRHS_CUDA(ctx, cudaGetLastError());
    prhs_status rc = prhs_decode_step(ctx, layer, step, sched, ctx->st_q, kv, batch, dout, nullptr, stream);
    if (rc != PRHS_OK) return rc;
    if (sync) PRHS_CUDA(ctx, cudaStreamSynchronize(st));
    return PRHS_OK;
  }
  PRHS_CUDA(ctx, cudaMemcpyAsync(ctx->st_q, host_q, qb, cudaMemcpyHostToDevice, st));
  PRHS_CUDA(ctx, cudaMemcpyAsync(ctx->st_k, host_new_k, kb, cudaMemcpyHostToDevice, st));
  PRHS_CUDA(ctx, cudaMemcpyAsync(ctx->st_v, host_new_v, kb, cudaMemcpyHostToDevice, st));
  PRHS_CUDA(ctx, cudaMemcpyAsync(const_cast<int32_t*>(kv->seq_lens), host_seq_lens, batch * sizeof(int32_t),
                                 cudaMemcpyHostToDevice, st));
  {
    LaunchScope ls(ctx, PRHS_KIND_MISC, st);
    append_rows_kernel<<<dim3(ctx->cfg.num_kv_heads, batch), 32, 0, st>>>(
        ctx->st_k, ctx->st_v, static_cast<__nv_bfloat16*>(const_cast<void*>(kv->k)),
        static_cast<__nv_bfloat16*>(const_cast<void*>(kv->v)), kv->stride_outer, kv->stride_head,
        kv->seq_lens, ctx->cfg.num_kv_heads);
  }
  PRHS_CUDA(ctx, cudaGetLastError());
  prhs_status rc = prhs_decode_step(ctx, layer, step, sched, ctx->st_q, kv, batch, ctx->st_out, nullptr, stream);
  if (rc != PRHS_OK) return rc;
  PRHS_CUDA(ctx, cudaMemcpyAsync(host_out, ctx->st_out, qb, cudaMemcpyDeviceToHost, st));
  if (sync) PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}
}  // namespace

prhs_status prhs_decode_step_host(prhs_ctx* ctx, int32_t layer, int32_t step, const prhs_schedule* sched,
                                  const void* host_q, const void* host_new_k, const void* host_new_v,
                                  const int32_t* host_seq_lens, const prhs_kv_view* kv, int32_t batch,
                                  void* host_out, void* stream) {
  return decode_step_host_impl(ctx, layer, step, sched, host_q, host_new_k, host_new_v, host_seq_lens, kv, batch,
                               host_out, stream, true);
}

prhs_status prhs_decode_step_host_async(prhs_ctx* ctx, int32_t layer, int32_t step, const prhs_schedule* sched,
                                        const void* host_q, const void* host_new_k, const void* host_new_v,
                                        const int32_t* host_seq_lens, const prhs_kv_view* kv, int32_t batch,
                                        void* host_out, void* stream) {
  return decode_step_host_impl(ctx, layer, step, sched, host_q, host_new_k, host_new_v, host_seq_lens, kv, batch,
                               host_out, stream, false);
}

prhs_status prhs_delta(prhs_ctx* ctx, const void* q, const prhs_kv_view* kv, const int32_t* idx,
                       const int32_t* count, int32_t idx_stride, int32_t batch, float* out_delta,
                       void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!q || !idx || !count || !out_delta) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  if (idx_stride < 1) return fail(ctx, PRHS_ERR_INVALID_ARG, "idx_stride must be >= 1");
  KvDev dv;
  int max_t;
  prhs_status rc = check_view(ctx, kv, batch, &dv, &max_t);
  if (rc != PRHS_OK) return rc;
  cudaStream_t st = as_stream(stream);
  int nchunks = 1;
  rc = launch_score(ctx, q, dv, batch, max_t, nullptr, nullptr, st, &nchunks);
  if (rc != PRHS_OK) return rc;
  const int n = batch * ctx->cfg.num_q_heads;
  {
    LaunchScope ls(ctx, PRHS_KIND_MISC, st);
    lse_reduce_kernel<<<(n + 127) / 128, 128, 0, st>>>(ctx->part_ml, nchunks, 0, dv.seq_lens,
                                                         ctx->cfg.num_q_heads, ctx->lse_full, n);
  }
  PRHS_CUDA(ctx, cudaGetLastError());
  return launch_attn(ctx, q, dv, idx, count, idx_stride, SetRef{}, idx_stride, batch, ctx->scratch_out,
                     ctx->lse_c, ctx->lse_full, out_delta, st, max_t);
}

prhs_status prhs_get_index_set(prhs_ctx* ctx, int32_t batch, int32_t* host_idx, int32_t* host_count,
                               void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (batch < 1 || batch > ctx->cfg.max_batch) return fail(ctx, PRHS_ERR_CAPACITY, "batch out of range");
  cudaStream_t st = as_stream(stream);
  const size_t n = (size_t)batch * ctx->cfg.num_q_heads;
  if (!ctx->last_set.star || batch != ctx->last_batch)
    return fail(ctx, PRHS_ERR_STATE, "no decode step to report (or a different batch)");
  prhs_status rc = launch_build(ctx, ctx->last_set, ctx->last_seq_lens, batch, ctx->idx, ctx->idx_cap,
                                ctx->count, st);
  if (rc != PRHS_OK) return rc;
  if (host_idx)
    PRHS_CUDA(ctx, cudaMemcpyAsync(host_idx, ctx->idx, n * ctx->idx_cap * sizeof(int), cudaMemcpyDeviceToHost, st));
  if (host_count)
    PRHS_CUDA(ctx, cudaMemcpyAsync(host_count, ctx->count, n * sizeof(int), cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}

prhs_status prhs_get_shared_set(prhs_ctx* ctx, int32_t layer, int32_t batch, int32_t* host_s_star,
                                int32_t* host_n_star, int32_t* host_s_hat, int32_t* host_n_hat,
                                void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (batch < 1 || batch > ctx->cfg.max_batch) return fail(ctx, PRHS_ERR_CAPACITY, "batch out of range");
  // groups are indexed with the layer_group of the schedule that last retrieved
  const int g = layer / ctx->last_layer_group;
  if (layer < 0 || g >= ctx->num_groups) return fail(ctx, PRHS_ERR_INVALID_ARG, "layer out of range");
  cudaStream_t st = as_stream(stream);
  const size_t n = (size_t)batch * ctx->cfg.num_q_heads;
  // the slot each unit used in the group's latest step (slot 0 without the cosine gate)
  std::vector<int> slot(n, 0);
  if (ctx->slots > 1 && ctx->gate_step[g] >= 0) {
    PRHS_CUDA(ctx, cudaMemcpyAsync(slot.data(), ctx->g_slot + unit_off(ctx, g), n * sizeof(int),
                                   cudaMemcpyDeviceToHost, st));
    PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  }
  const size_t mk = ctx->cfg.max_k, hc = ctx->shat_cap, SL = ctx->slots;
  const size_t share = (size_t)std::max(ctx->last_share_gq, 1);   // group-shared sets live with the group's first head
  for (size_t u = 0; u < n; ++u) {
    const size_t e = (u - u % share) * SL + (size_t)slot[u];
    if (host_s_star)
      PRHS_CUDA(ctx, cudaMemcpyAsync(host_s_star + u * mk, ctx->sstar_desc + state_off(ctx, g, mk) + e * mk,
                                     mk * sizeof(int), cudaMemcpyDeviceToHost, st));
    if (host_n_star)
      PRHS_CUDA(ctx, cudaMemcpyAsync(host_n_star + u, ctx->n_star + state_off(ctx, g, 1) + e, sizeof(int),
                                     cudaMemcpyDeviceToHost, st));
    if (host_s_hat)
      PRHS_CUDA(ctx, cudaMemcpyAsync(host_s_hat + u * hc, ctx->shat_asc + state_off(ctx, g, hc) + e * hc,
                                     hc * sizeof(int), cudaMemcpyDeviceToHost, st));
    if (host_n_hat)
      PRHS_CUDA(ctx, cudaMemcpyAsync(host_n_hat + u, ctx->n_hat + state_off(ctx, g, 1) + e, sizeof(int),
                                     cudaMemcpyDeviceToHost, st));
  }
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}

prhs_status prhs_get_gate(prhs_ctx* ctx, int32_t layer, int32_t batch, int32_t* host_need,
                          int32_t* host_ref, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (batch < 1 || batch > ctx->cfg.max_batch) return fail(ctx, PRHS_ERR_CAPACITY, "batch out of range");
  const int g = layer / ctx->last_layer_group;
  if (layer < 0 || g >= ctx->num_groups) return fail(ctx, PRHS_ERR_INVALID_ARG, "layer out of range");
  if (ctx->gate_step[g] < 0) return fail(ctx, PRHS_ERR_STATE, "no gated step has run for this layer group");
  cudaStream_t st = as_stream(stream);
  const size_t n = (size_t)batch * ctx->cfg.num_q_heads;
  if (host_need)
    PRHS_CUDA(ctx, cudaMemcpyAsync(host_need, ctx->g_need + unit_off(ctx, g), n * sizeof(int),
                                   cudaMemcpyDeviceToHost, st));
  if (host_ref)
    PRHS_CUDA(ctx, cudaMemcpyAsync(host_ref, ctx->g_ref + unit_off(ctx, g), n * sizeof(int),
                                   cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}

prhs_status prhs_get_scores(prhs_ctx* ctx, int32_t batch, float* host_scores, void* stream) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (!host_scores) return fail(ctx, PRHS_ERR_INVALID_ARG, "NULL pointer");
  if (batch < 1 || batch > ctx->cfg.max_batch) return fail(ctx, PRHS_ERR_CAPACITY, "batch out of range");
  cudaStream_t st = as_stream(stream);
  PRHS_CUDA(ctx, cudaMemcpyAsync(host_scores, ctx->scores,
                                 (size_t)batch * ctx->cfg.num_q_heads * ctx->ld * sizeof(float),
                                 cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  return PRHS_OK;
}

const char* prhs_kernel_kind_name(int32_t kind) {
  static const char* names[PRHS_KERNEL_KINDS] = {"score", "select", "build_set", "attn_sparse",
                                                 "attn_dense", "misc"};
  return (kind >= 0 && kind < PRHS_KERNEL_KINDS) ? names[kind] : "?";
}

prhs_status prhs_profile_begin(prhs_ctx* ctx, int32_t max_launches) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  if (max_launches < 1 || max_launches > (1 << 20))
    return fail(ctx, PRHS_ERR_INVALID_ARG, "max_launches out of range");
  while ((int)ctx->prof.size() < max_launches) {
    prhs_ctx::ProfRec r;
    r.kind = 0;
    PRHS_CUDA(ctx, cudaEventCreate(&r.a));
    cudaError_t e = cudaEventCreate(&r.b);
    if (e != cudaSuccess) {
      cudaEventDestroy(r.a);
      return fail(ctx, PRHS_ERR_CUDA, cudaGetErrorString(e));
    }
    ctx->prof.push_back(r);
  }
  ctx->prof_used = 0;
  ctx->prof_on = true;
  return PRHS_OK;
}

prhs_status prhs_profile_end(prhs_ctx* ctx, void* stream, float* host_ms_per_kind,
                             int64_t* host_launches_per_kind) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  ctx->prof_on = false;
  PRHS_CUDA(ctx, cudaStreamSynchronize(as_stream(stream)));
  for (int k = 0; k < PRHS_KERNEL_KINDS; ++k) {
    if (host_ms_per_kind) host_ms_per_kind[k] = 0.f;
    if (host_launches_per_kind) host_launches_per_kind[k] = 0;
  }
  for (int i = 0; i < ctx->prof_used; ++i) {
    float ms = 0.f;
    PRHS_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->prof[i].a, ctx->prof[i].b));
    if (host_ms_per_kind) host_ms_per_kind[ctx->prof[i].kind] += ms;
    if (host_launches_per_kind) host_launches_per_kind[ctx->prof[i].kind] += 1;
  }
  ctx->prof_used = 0;
  return PRHS_OK;
}

prhs_status prhs_check(prhs_ctx* ctx, void* stream, uint32_t* out_flags) {
  if (!ctx) return PRHS_ERR_INVALID_ARG;
  cudaStream_t st = as_stream(stream);
  uint32_t f = 0;
  PRHS_CUDA(ctx, cudaMemcpyAsync(&f, ctx->flags, sizeof(f), cudaMemcpyDeviceToHost, st));
  PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  PRHS_CUDA(ctx, cudaGetLastError());
  if (out_flags) *out_flags = f;
  if (f) {
    PRHS_CUDA(ctx, cudaMemsetAsync(ctx->flags, 0, sizeof(uint32_t), st));
    PRHS_CUDA(ctx, cudaStreamSynchronize(st));
  }
  if (f & (PRHS_FLAG_BAD_INDEX | PRHS_FLAG_BAD_PAGE | PRHS_FLAG_TIMEOUT)) {
    char buf[96];
    snprintf(buf, sizeof buf, "device flag word 0x%x", f);
    return fail(ctx, PRHS_ERR_DEVICE_FLAG, buf);
  }
  return PRHS_OK;
}

}  // extern "C"
