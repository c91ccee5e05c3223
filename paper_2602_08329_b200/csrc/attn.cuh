// Index-set builder (Sec. 4.1 critical set; Def. 3.2 key-value sharing) and the gathered
// split-K flash-decoding attention over the selected rows (Def. 3.1), with its merge.
#pragma once
#include "common.cuh"

namespace prhs {

// ------------------------------------------------------------------ index-set builder
// C = [0, min(S0,t)) U M U [max(0,t-W), t), ascending and unique.  M is ascending and
// unique already, so the union is: the sink run, M clipped to [S0', wlo), the window run.
// One CTA per (sequence, query head).
__global__ void __launch_bounds__(128)
build_set_kernel(SetRef ref, const int* __restrict__ seq_lens, int num_q_heads,
                 int* __restrict__ out_idx, int idx_stride, int* __restrict__ out_count) {
  const int unit = blockIdx.x;
  const int b = unit / num_q_heads;
  const int t = __ldg(seq_lens + b);
  int nm, mstride;
  const int* M = middle_of(ref, unit, &nm, &mstride);
  const int s0 = min(ref.sinks, t);
  const int vis_lo = max(s0, psaw_start(ref.psaw_c, t));  // first visible non-sink position
  const int wlo = max(max(t - ref.window, 0), vis_lo);
  // M is ascending: the number of entries below a bound is the position of the bound.  Count
  // in parallel (one coalesced pass) instead of a binary search of dependent cold loads.
  __shared__ int sh_lo, sh_hi;
  if (threadIdx.x == 0) { sh_lo = 0; sh_hi = 0; }
  __syncthreads();
  int c0 = 0, c1 = 0;
  for (int i = threadIdx.x; i < nm; i += blockDim.x) {
    const int x = __ldg(M + i);
    c0 += x < vis_lo;
    c1 += x < wlo;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    c0 += __shfl_xor_sync(0xffffffffu, c0, off);
    c1 += __shfl_xor_sync(0xffffffffu, c1, off);
  }
  if ((threadIdx.x & 31) == 0) { atomicAdd(&sh_lo, c0); atomicAdd(&sh_hi, c1); }
  __syncthreads();
  const int lo = sh_lo, hi = max(sh_hi, sh_lo);
  const int nmid = hi - lo;
  const int total = s0 + nmid + (t - wlo);
  int* out = out_idx + (long long)unit * idx_stride;
  for (int j = threadIdx.x; j < total && j < idx_stride; j += blockDim.x) {
    int v;
    if (j < s0) v = j;
    else if (j < s0 + nmid) v = __ldg(M + lo + (j - s0));
    else v = wlo + (j - s0 - nmid);
    out[j] = v;
  }
  if (threadIdx.x == 0) out_count[unit] = min(total, idx_stride);
}

// ------------------------------------------------------------ gathered / dense attention
constexpr int kPartStride = kHeadDim + 4;         // o[128] (unnormalised), m, l, l~ per split (+ padding)

struct AttnParams {
  const __nv_bfloat16* q;   // [B][Hq][128]
  KvDev kv;
  const int* idx;           // [B][Hq][idx_stride] or nullptr
  const int* count;         // [B][Hq] (with idx)
  int idx_stride;
  // fused index-set builder (used when idx == nullptr and set.star != nullptr): the list is
  // [0, s0) ++ M clipped to [vis_lo, wlo) ++ [wlo, t) with M the unit's stored middle set
  SetRef set;
  // idx == nullptr and set.star == nullptr: all positions [0, t) (dense baseline)
  int num_q_heads, group_size;
  int splits;
  float* partials;          // [B][Hq][splits][kPartStride]: o, m, l, l~ (see below)
  unsigned int* tickets;    // [B][Hq], zero on entry, zero again on exit
  __nv_bfloat16* out;       // [B][Hq][128]
  float* out_lse;           // [B][Hq] or nullptr
  const float* lse_full;    // [B][Hq] or nullptr
  float* out_delta;         // [B][Hq] or nullptr: 1 - exp(lse - lse_full)
  uint32_t* flags;
  // cosine-gated steps launch the attention twice, for the heads that share (beside the retrieval
  // of the others) and for the heads that retrieved (after it): need_mode 1 = only units with
  // need[unit] == 0, 2 = only units with need[unit] != 0, 0 = every unit
  const int* need;
  int need_mode;
};

// ---------------------------------------------------------------- cp.async helpers
constexpr uint32_t kBadRow = 0xffffffffu;

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes)
               : "memory");
}
__device__ __forceinline__ void cp_async_16_full(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Where list entry j of a (b, h) unit lives: an explicit list, the fused sinks/middle/window
// description, or the identity (dense).
struct ListDesc {
  const int* list;   // explicit list, or the middle set M in fused mode
  int fused;         // 1: entry j < s0 -> j; j < s0 + nmid -> list[lo + j - s0]; else wlo + ...
  int s0, nmid, lo, wlo;
  int count;
};

// Entry j of a unit's list, unchecked: for a stored middle entry this is a load whose result the
// caller must not look at before it needs it (the row-id pipeline issues it a step ahead).
__device__ __forceinline__ int list_entry(const ListDesc& ld, int j, int end) {
  if (j >= end) return -1;
  if (ld.fused) {
    if (j < ld.s0) return j;
    if (j < ld.s0 + ld.nmid) return __ldg(ld.list + ld.lo + (j - ld.s0));
    return ld.wlo + (j - ld.s0 - ld.nmid);
  }
  return ld.list ? __ldg(ld.list + j) : j;
}

// The entry checked (this consumes the load): the position if it is a real row of the sequence,
// else -1.  A stored middle entry that has moved into the window is left out silently (the window
// part of the list covers it); a position outside [0, t) is recorded as an anomaly.
__device__ __forceinline__ int checked_entry(const ListDesc& ld, int pos, int j, int end, int t, uint32_t* flags) {
  if (j >= end) return -1;
  if (ld.fused && j >= ld.s0 && j < ld.s0 + ld.nmid && pos >= ld.wlo) return -1;
  if ((unsigned)pos >= (unsigned)t) {
    atomicOr(flags, kFlagBadIndex);
    return -1;
  }
  return pos;
}

// Per-warp set-up of the list descriptor (all 32 lanes call it).  In fused mode the middle part is
// M without its entries below vis_lo: dilation can push at most r entries below S0, so a look at
// the first 32 entries (a load that does not wait for the set's size) settles it; a longer overlap
// (a sliding window start that moved past many entries) falls back to a full scan.  Entries of M
// that have moved into the window since the set was stored (again at most r, at its end) stay
// in the list and are masked where they are read: counting them would cost one more round of
// dependent loads before the first row can be requested.
__device__ __forceinline__ ListDesc make_list_desc(const AttnParams& p, int unit, int t) {
  ListDesc d;
  const int lane = threadIdx.x & 31;
  d.fused = 0; d.s0 = 0; d.nmid = 0; d.lo = 0; d.wlo = 0;
  if (p.idx) {
    d.list = p.idx + (long long)unit * p.idx_stride;
    d.count = min(__ldg(p.count + unit), p.idx_stride);
  } else if (p.set.star) {
    int nm, mstride;
    const int* M = middle_of(p.set, unit, &nm, &mstride);
    const int s0 = min(p.set.sinks, t);
    const int vis_lo = max(s0, psaw_start(p.set.psaw_c, t));
    const int wlo = max(max(t - p.set.window, 0), vis_lo);
    const int head = lane < mstride ? __ldg(M + lane) : 0x7fffffff;     // does not depend on nm
    int lo = __popc(__ballot_sync(0xffffffffu, lane < nm && head < vis_lo));
    if (lo == 32) {                     // a sliding window start far into the set: count everything
      int c0 = 0;
      for (int i = lane; i < nm; i += 32) c0 += __ldg(M + i) < vis_lo;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) c0 += __shfl_xor_sync(0xffffffffu, c0, off);
      lo = c0;
    }
    d.list = M; d.fused = 1; d.s0 = s0; d.lo = lo; d.wlo = wlo;
    d.nmid = max(nm - lo, 0);
    d.count = s0 + d.nmid + (t - wlo);
  } else {
    d.list = nullptr;
    d.count = t;
  }
  return d;
}

// ------------------------------------------- gathered attention, tensor-core pipeline (sm_100a)
// The same warp-private cp.async pipeline, with the arithmetic moved to mma.sync m16n8k16
// (bf16 in, fp32 accumulate) so that a gathered row costs about a dozen warp instructions
// instead of about fifty.  A stage is 16 list entries: a K tile and a V tile of [16][128]
// bf16, 16-byte chunk c of row r stored at chunk c ^ (r & 7) (ldmatrix reads conflict-free).
//   S = Q K^T : A = the query as row 0 of a 16-row tile (rows 1..15 zero), B = K tile
//               (ldmatrix), 2 n-tiles x 8 k-steps; lanes 0-3 end up with the 16 logits.
//   O += P V  : A = P from the S accumulators (row 0 only), B = V tile (ldmatrix.trans),
//               16 n-tiles x 1 k-step; lanes 0-3 hold the 128 output columns.
// Index sets are per query head, so only one of the 16 tile rows carries data; the tensor
// cores are used for their instruction economy, not their FLOPs.
// The weights enter the P V product rounded to bf16.  Two sums of them are kept: l, of the fp32
// weights, gives the log-sum-exp (and through it delta) at full precision; l~, of the weights
// as rounded, divides the output, so that the output is a convex combination of the value rows
// with consistently normalised weights (where one key dominates, its weight stays 1 instead of
// carrying the rounding error of its bf16 image).
constexpr int kTWarps = 4;
constexpr int kTThreads = kTWarps * 32;
constexpr int kTStageRows = 16;
constexpr int kTStages = 3;
constexpr int kTTileBytes = kTStageRows * kRowBytes;                 // 4 KB
constexpr int kTStageBytes = 2 * kTTileBytes;                        // K tile + V tile
constexpr int kTSmemBytes = kTWarps * kTStages * kTStageBytes;       // 96 KB

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A * B with A rows 8..15 zero (a1 = a3 = 0): only accumulator rows 0..7 are live.
__device__ __forceinline__ void mma_bf16_row0(float& d0, float& d1, float& z0, float& z1, uint32_t a0,
                                              uint32_t a2, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d0), "+f"(d1), "+f"(z0), "+f"(z1)
      : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_bf16_full(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

template <int kValue>
struct SlotC { static constexpr int value = kValue; };    // a ring slot known at compile time

__global__ void __launch_bounds__(kTThreads) gather_attn_mma_kernel(AttnParams p) {
  extern __shared__ __align__(128) unsigned char g_smem[];
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int unit = b * p.num_q_heads + h;
  if (p.need_mode != 0 && ((__ldg(p.need + unit) != 0) != (p.need_mode == 2))) return;   // the other launch's unit
  const int kvh = h / p.group_size;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int t = __ldg(p.kv.seq_lens + b);
  const ListDesc ld = make_list_desc(p, unit, t);
  const int cnt = ld.count;
  int per = (cnt + p.splits * kTWarps - 1) / (p.splits * kTWarps);
  per = (per + kTStageRows - 1) & ~(kTStageRows - 1);
  const int start = min((split * kTWarps + warp) * per, cnt);
  const int end = min(start + per, cnt);
  const int nstages = (end - start + kTStageRows - 1) / kTStageRows;
  const uint32_t outer_rows = (uint32_t)(p.kv.stride_outer >> 7);
  const uint32_t head_rows = (uint32_t)(p.kv.stride_head >> 7);
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(g_smem) + warp * (kTStages * kTStageBytes);

  // A fragments of the query: row 0 of the tile lives in lanes 0-3 (g == 0)
  uint32_t aq0[8], aq2[8];
  {
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q + (long long)unit * kHeadDim);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      aq0[ks] = g == 0 ? __ldg(q32 + ks * 8 + tg) : 0u;
      aq2[ks] = g == 0 ? __ldg(q32 + ks * 8 + 4 + tg) : 0u;
    }
  }
  // O^T += V^T P^T: the 128 output columns sit on the M rows of eight 16 x 8 tiles whose column 0
  // is live (lanes with tg == 0 hold columns 16 mt + g and 16 mt + g + 8 in o[mt][0], o[mt][2])
  float o[8][4];
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) { o[mt][0] = 0.f; o[mt][1] = 0.f; o[mt][2] = 0.f; o[mt][3] = 0.f; }
  float m = -INFINITY, l = 0.f, lt = 0.f;     // lt: the sum of the weights as rounded to bf16

  // Row-id pipeline, 32 list entries (two stages) per step, one entry per lane.  Each level is
  // produced one step before it is consumed, so that no load is waited for where it is issued:
  //   pos2 : raw list entry of group G+2 (a load from the list, unchecked)
  //   pos1 / pg1 : checked position of group G+1 and, for a paged cache, its raw page id (a load)
  //   rid_a : final row id of group G, the one being issued
  auto list_pos = [&](int grp) -> int { return list_entry(ld, start + grp * 32 + lane, end); };
  auto check_pos = [&](int pos, int grp) -> int {      // consumes the list load
    return checked_entry(ld, pos, start + grp * 32 + lane, end, t, p.flags);
  };
  const bool paged = p.kv.page_table != nullptr;
  auto page_of = [&](int pos) -> int {                 // issues the page-table load
    if (!paged || pos < 0) return 0;
    return __ldg(p.kv.page_table + (long long)b * p.kv.page_table_stride + (pos >> kPageShift));
  };
  auto row_id = [&](int pos, int page) -> uint32_t {   // consumes the page-table load
    if (pos < 0) return kBadRow;
    if (paged) {
      if ((unsigned)page >= (unsigned)p.kv.num_pages) {
        atomicOr(p.flags, kFlagBadPage);
        return kBadRow;
      }
      return (uint32_t)page * outer_rows + (uint32_t)kvh * head_rows + (uint32_t)(pos & 15);
    }
    return (uint32_t)b * outer_rows + (uint32_t)kvh * head_rows + (uint32_t)pos;
  };
  int pos1 = check_pos(list_pos(0), 0);
  int pg1 = page_of(pos1);
  uint32_t rid_a = row_id(pos1, pg1);
  // validity of the 32 entries of the group being issued, one bit per lane; invalid entries
  // point at row 0 (a valid address) and are copied with size 0 (zero fill)
  uint32_t valid_a = __ballot_sync(0xffffffffu, rid_a != kBadRow);
  if (rid_a == kBadRow) rid_a = 0u;
  pos1 = check_pos(list_pos(1), 1);
  pg1 = page_of(pos1);
  int pos2 = list_pos(2);

  // The copy of row r of a stage: lane p (0-15: K row, 16-31: V row) fills 16-byte position p of the
  // row with the source chunk p ^ (r & 7), which is the XOR swizzle ldmatrix reads.  Written this
  // way the destination of a lane is the same in every row and the eight source offsets are
  // loop invariants: a row costs a shuffle, one multiply-add and the copy.
  const __nv_bfloat16* srcx[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) srcx[k] = (lane < 16 ? p.kv.k : p.kv.v) + ((((uint32_t)lane & 15u) ^ (uint32_t)k) << 3);
  const uint32_t dst_lane = (lane < 16 ? 0u : (uint32_t)kTTileBytes) + (((uint32_t)lane & 15u) << 4);
  uint32_t vmv[kTStages];              // 16 validity bits per ring slot (slots are compile-time below)
#pragma unroll
  for (int k = 0; k < kTStages; ++k) vmv[k] = 0u;

  auto issue = [&](int j, auto slot_c) {
    constexpr int kSlot = decltype(slot_c)::value;
    if (j < nstages) {
      if (j > 0 && (j & 1) == 0) {     // step the row-id pipeline
        const int grp = j >> 1;
        rid_a = row_id(pos1, pg1);
        valid_a = __ballot_sync(0xffffffffu, rid_a != kBadRow);
        if (rid_a == kBadRow) rid_a = 0u;
        pos1 = check_pos(pos2, grp + 1);
        pg1 = page_of(pos1);
        pos2 = list_pos(grp + 2);
      }
      // the 16 entries of this stage, brought to lanes 0-15 (odd stages hold them in lanes 16-31)
      const uint32_t rid_cur = __shfl_sync(0xffffffffu, rid_a, (lane + ((j & 1) << 4)) & 31);
      const uint32_t slot = ring + (uint32_t)kSlot * kTStageBytes + dst_lane;
      const uint32_t vm = (valid_a >> ((j & 1) * kTStageRows)) & 0xffffu;
      if (vm == 0xffffu) {             // the common case: 16 real rows
#pragma unroll
        for (int r = 0; r < kTStageRows; ++r) {
          const uint32_t rid = __shfl_sync(0xffffffffu, rid_cur, r);
          cp_async_16_full(slot + r * kRowBytes, srcx[r & 7] + (size_t)rid * kHeadDim);
        }
      } else {
#pragma unroll
        for (int r = 0; r < kTStageRows; ++r) {
          const uint32_t rid = __shfl_sync(0xffffffffu, rid_cur, r);
          cp_async_16(slot + r * kRowBytes, srcx[r & 7] + (size_t)rid * kHeadDim, ((vm >> r) & 1u) ? 16 : 0);
        }
      }
      vmv[kSlot] = vm;
    }
    cp_async_commit();
  };

  issue(0, SlotC<0>{});
  issue(1, SlotC<1>{});
  static_assert(kTStages == 3, "the stage loop below is unrolled over three ring slots");

  const float sc = kScale * kLog2e;
  // ldmatrix lane roles
  const int lm_mi = lane >> 3, lm_r = lane & 7;
  const int vrow = (lm_mi & 1) * 8 + lm_r;
  // One stage: wait for its copies, refill the slot two stages ahead, S = Q K^T, softmax, O += P V.
  auto stage = [&](int i, auto slot_c) {
    constexpr int kSlot = decltype(slot_c)::value;
    cp_async_wait<kTStages - 2>();
    __syncwarp();
    const uint32_t vm = vmv[kSlot];
    issue(i + kTStages - 1, SlotC<(kSlot + kTStages - 1) % kTStages>{});
    const uint32_t kt = ring + (uint32_t)kSlot * kTStageBytes;
    const uint32_t vt = kt + kTTileBytes;
    // ---- S = Q K^T : all K fragments first, then the two accumulator chains interleaved
    uint32_t bk[2][4][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int row = nt * 8 + lm_r;
#pragma unroll
      for (int pp = 0; pp < 4; ++pp)
        ldmatrix_x4(bk[nt][pp], kt + row * kRowBytes + (((4 * pp + lm_mi) ^ (row & 7)) << 4));
    }
    // (the dead accumulator rows 8..15 get registers of their own per chain: one pair shared by
    // all MMAs would chain them all through it)
    float s[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    float zq[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
#pragma unroll
    for (int pp = 0; pp < 4; ++pp) {
      mma_bf16_row0(s[0][0], s[0][1], zq[0][0], zq[0][1], aq0[2 * pp], aq2[2 * pp], bk[0][pp][0], bk[0][pp][1]);
      mma_bf16_row0(s[1][0], s[1][1], zq[1][0], zq[1][1], aq0[2 * pp], aq2[2 * pp], bk[1][pp][0], bk[1][pp][1]);
      mma_bf16_row0(s[0][0], s[0][1], zq[0][0], zq[0][1], aq0[2 * pp + 1], aq2[2 * pp + 1], bk[0][pp][2], bk[0][pp][3]);
      mma_bf16_row0(s[1][0], s[1][1], zq[1][0], zq[1][1], aq0[2 * pp + 1], aq2[2 * pp + 1], bk[1][pp][2], bk[1][pp][3]);
    }
    // the first half of the V fragments, fetched under the softmax arithmetic
    uint32_t bv[4][4];
#pragma unroll
    for (int np = 0; np < 4; ++np)
      ldmatrix_x4_trans(bv[np], vt + vrow * kRowBytes + (((2 * np + (lm_mi >> 1)) ^ (vrow & 7)) << 4));
    // ---- online softmax on the 16 logits held by lanes 0-3.  The reference exponent m only
    // moves when a logit exceeds it by more than 8 (weights stay below 2^8): the common
    // stage costs one warp vote instead of a cross-lane maximum.
    float s0 = -INFINITY, s1 = -INFINITY, s2 = -INFINITY, s3 = -INFINITY;
    if (g == 0) {
      if ((vm >> (2 * tg)) & 1u) s0 = s[0][0] * sc;
      if ((vm >> (2 * tg + 1)) & 1u) s1 = s[0][1] * sc;
      if ((vm >> (8 + 2 * tg)) & 1u) s2 = s[1][0] * sc;
      if ((vm >> (9 + 2 * tg)) & 1u) s3 = s[1][1] * sc;
    }
    float mx = fmaxf(fmaxf(s0, s1), fmaxf(s2, s3));
    if (__any_sync(0xffffffffu, mx > m + 8.f)) {
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float mn = fmaxf(m, __shfl_sync(0xffffffffu, mx, 0));
      const float corr = exp2f(m - mn);     // m = -inf on the first real stage: corr = 0
      m = mn;
      l *= corr;
      lt *= corr;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= corr; o[mt][1] *= corr; o[mt][2] *= corr; o[mt][3] *= corr; }
    }
    if (m != -INFINITY) {              // warp-uniform; false only while every row so far was invalid
      const float p0 = exp2f(s0 - m), p1 = exp2f(s1 - m), p2 = exp2f(s2 - m), p3 = exp2f(s3 - m);
      l += (p0 + p1) + (p2 + p3);
      const uint32_t ap0 = pack_bf16x2(p0, p1), ap2 = pack_bf16x2(p2, p3);
      lt += (bf_lo(ap0) + bf_hi(ap0)) + (bf_lo(ap2) + bf_hi(ap2));
      // ---- O^T += V^T P^T: the transposed V fragments of 16 columns are the A operand of one
      // 16 x 16 tile (rows g / g + 8 x keys 2tg.. / 2tg+8..), the weights the B operand's column 0:
      // eight independent MMAs per stage
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) mma_bf16_full(o[mt], bv[mt][0], bv[mt][2], bv[mt][1], bv[mt][3], ap0, ap2);
#pragma unroll
      for (int np = 4; np < 8; ++np)
        ldmatrix_x4_trans(bv[np - 4], vt + vrow * kRowBytes + (((2 * np + (lm_mi >> 1)) ^ (vrow & 7)) << 4));
#pragma unroll
      for (int mt = 4; mt < 8; ++mt)
        mma_bf16_full(o[mt], bv[mt - 4][0], bv[mt - 4][2], bv[mt - 4][1], bv[mt - 4][3], ap0, ap2);
    }
  };
  {
    int i = 0;
    for (; i + 2 < nstages; i += 3) {
      stage(i, SlotC<0>{});
      stage(i + 1, SlotC<1>{});
      stage(i + 2, SlotC<2>{});
    }
    if (i < nstages) stage(i, SlotC<0>{});
    if (i + 1 < nstages) stage(i + 1, SlotC<1>{});
  }
  cp_async_wait<0>();
  l += __shfl_xor_sync(0xffffffffu, l, 1);
  l += __shfl_xor_sync(0xffffffffu, l, 2);
  lt += __shfl_xor_sync(0xffffffffu, lt, 1);
  lt += __shfl_xor_sync(0xffffffffu, lt, 2);

  // ---- combine the warps of this CTA (lanes with tg == 0 hold columns 16*mt + g and 16*mt + g + 8)
  __shared__ __align__(16) float sm_o[kTWarps][kHeadDim];       // written as float2
  __shared__ float sm_m[kTWarps], sm_l[kTWarps], sm_lt[kTWarps];
  __shared__ bool is_last;
  if (tg == 0) {
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      sm_o[warp][16 * mt + g] = o[mt][0];
      sm_o[warp][16 * mt + g + 8] = o[mt][2];
    }
  }
  if (lane == 0) { sm_m[warp] = m; sm_l[warp] = l; sm_lt[warp] = lt; }
  __syncthreads();
  {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kTWarps; ++w) M = fmaxf(M, sm_m[w]);
    float acc = 0.f, L = 0.f, Lt = 0.f;
    if (M != -INFINITY) {
#pragma unroll
      for (int w = 0; w < kTWarps; ++w) {
        const float scw = exp2f(sm_m[w] - M);
        acc = fmaf(sm_o[w][tid], scw, acc);
        L = fmaf(sm_l[w], scw, L);
        Lt = fmaf(sm_lt[w], scw, Lt);
      }
    }
    if (p.splits == 1) {
      p.out[(long long)unit * kHeadDim + tid] = __float2bfloat16_rn(Lt > 0.f ? acc / Lt : 0.f);
      if (tid == 0) {
        const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
        if (p.out_lse) p.out_lse[unit] = lse;
        if (p.out_delta) p.out_delta[unit] = L > 0.f ? -expm1f(lse - p.lse_full[unit]) : 1.f;
      }
      return;
    }
    float* part = p.partials + ((long long)unit * p.splits + split) * kPartStride;
    part[tid] = acc;
    if (tid == 0) { part[kHeadDim] = M; part[kHeadDim + 1] = L; part[kHeadDim + 2] = Lt; }
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned int ticket = atomicAdd(p.tickets + unit, 1u);
    is_last = (ticket == (unsigned int)p.splits - 1u);
    if (is_last) p.tickets[unit] = 0u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  const float* base = p.partials + (long long)unit * p.splits * kPartStride;
  float M = -INFINITY;
  for (int sp = 0; sp < p.splits; ++sp) M = fmaxf(M, __ldcg(base + sp * kPartStride + kHeadDim));
  float acc = 0.f, L = 0.f, Lt = 0.f;
  if (M != -INFINITY) {
    for (int sp = 0; sp < p.splits; ++sp) {
      const float scw = exp2f(__ldcg(base + sp * kPartStride + kHeadDim) - M);
      acc = fmaf(__ldcg(base + sp * kPartStride + tid), scw, acc);
      L = fmaf(__ldcg(base + sp * kPartStride + kHeadDim + 1), scw, L);
      Lt = fmaf(__ldcg(base + sp * kPartStride + kHeadDim + 2), scw, Lt);
    }
  }
  p.out[(long long)unit * kHeadDim + tid] = __float2bfloat16_rn(Lt > 0.f ? acc / Lt : 0.f);
  if (tid == 0) {
    const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
    if (p.out_lse) p.out_lse[unit] = lse;
    if (p.out_delta) p.out_delta[unit] = L > 0.f ? -expm1f(lse - p.lse_full[unit]) : 1.f;
  }
}

// ---------------------------------------------------- dense flash-decode baseline (Eq. 2)
// Attention over every position [0, t): K and V of a KV head are read ONCE for all the
// query heads of its group, which sit on the 16 rows of the MMA tile (head j of the group =
// row j).  Same warp-private cp.async ring, swizzle and fragment plumbing as the gathered
// kernel; rows are consecutive, so the copies need no index list, and a 16-row stage that
// starts on a multiple of 16 lies in one page of a paged cache.
// grid (splits, Hkv, B).  Partials, tickets and outputs are per query head, as above.
// One 16-row stage of grouped attention: S = Q K^T for the heads on tile rows g and g + 8,
// online softmax per row with a lazy reference exponent, O += P V.  v0..v3 say which of this
// lane's four keys (rows 2tg, 2tg+1, 8+2tg, 9+2tg of the stage) are real.
__device__ __forceinline__ void group_stage(uint32_t kt, uint32_t vt, const uint32_t (&aq)[8][4], bool v0, bool v1,
                                            bool v2, bool v3, float (&o)[16][4], float& m0, float& l0, float& m1,
                                            float& l1, float& lt0, float& lt1) {
  const int lane = threadIdx.x & 31;
  const int lm_mi = lane >> 3, lm_r = lane & 7;
  const int vrow = (lm_mi & 1) * 8 + lm_r;
  const float sc = kScale * kLog2e;
  float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
  for (int pp = 0; pp < 4; ++pp) {
    uint32_t bk0[4], bk1[4];
    ldmatrix_x4(bk0, kt + lm_r * kRowBytes + (((4 * pp + lm_mi) ^ (lm_r & 7)) << 4));
    ldmatrix_x4(bk1, kt + (8 + lm_r) * kRowBytes + (((4 * pp + lm_mi) ^ (lm_r & 7)) << 4));
    mma_bf16_full(s[0], aq[2 * pp][0], aq[2 * pp][1], aq[2 * pp][2], aq[2 * pp][3], bk0[0], bk0[1]);
    mma_bf16_full(s[1], aq[2 * pp][0], aq[2 * pp][1], aq[2 * pp][2], aq[2 * pp][3], bk1[0], bk1[1]);
    mma_bf16_full(s[0], aq[2 * pp + 1][0], aq[2 * pp + 1][1], aq[2 * pp + 1][2], aq[2 * pp + 1][3], bk0[2], bk0[3]);
    mma_bf16_full(s[1], aq[2 * pp + 1][0], aq[2 * pp + 1][1], aq[2 * pp + 1][2], aq[2 * pp + 1][3], bk1[2], bk1[3]);
  }
  float x[2][4];   // [row half][key]
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    x[hh][0] = v0 ? s[0][2 * hh] * sc : -INFINITY;
    x[hh][1] = v1 ? s[0][2 * hh + 1] * sc : -INFINITY;
    x[hh][2] = v2 ? s[1][2 * hh] * sc : -INFINITY;
    x[hh][3] = v3 ? s[1][2 * hh + 1] * sc : -INFINITY;
  }
  // ---- online softmax per row (lazy reference exponent, as in the gathered kernel)
  float mx0 = fmaxf(fmaxf(x[0][0], x[0][1]), fmaxf(x[0][2], x[0][3]));
  float mx1 = fmaxf(fmaxf(x[1][0], x[1][1]), fmaxf(x[1][2], x[1][3]));
  if (__any_sync(0xffffffffu, mx0 > m0 + 8.f || mx1 > m1 + 8.f)) {
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
    const float c0 = (n0 == -INFINITY) ? 1.f : exp2f(m0 - n0);
    const float c1 = (n1 == -INFINITY) ? 1.f : exp2f(m1 - n1);
    m0 = n0; m1 = n1;
    l0 *= c0; l1 *= c1;
    lt0 *= c0; lt1 *= c1;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { o[nt][0] *= c0; o[nt][1] *= c0; o[nt][2] *= c1; o[nt][3] *= c1; }
  }
  float pw[2][4];
#pragma unroll
  for (int k4 = 0; k4 < 4; ++k4) {
    pw[0][k4] = (m0 == -INFINITY) ? 0.f : exp2f(x[0][k4] - m0);
    pw[1][k4] = (m1 == -INFINITY) ? 0.f : exp2f(x[1][k4] - m1);
  }
  l0 += (pw[0][0] + pw[0][1]) + (pw[0][2] + pw[0][3]);
  l1 += (pw[1][0] + pw[1][1]) + (pw[1][2] + pw[1][3]);
  const uint32_t a0 = pack_bf16x2(pw[0][0], pw[0][1]), a1 = pack_bf16x2(pw[1][0], pw[1][1]);
  const uint32_t a2 = pack_bf16x2(pw[0][2], pw[0][3]), a3 = pack_bf16x2(pw[1][2], pw[1][3]);
  lt0 += (bf_lo(a0) + bf_hi(a0)) + (bf_lo(a2) + bf_hi(a2));      // the weights as the MMA sees them
  lt1 += (bf_lo(a1) + bf_hi(a1)) + (bf_lo(a3) + bf_hi(a3));
  // ---- O += P V
#pragma unroll
  for (int np = 0; np < 8; ++np) {
    uint32_t bv[4];
    ldmatrix_x4_trans(bv, vt + vrow * kRowBytes + (((2 * np + (lm_mi >> 1)) ^ (vrow & 7)) << 4));
    mma_bf16_full(o[2 * np], a0, a1, a2, a3, bv[0], bv[1]);
    mma_bf16_full(o[2 * np + 1], a0, a1, a2, a3, bv[2], bv[3]);
  }
}

// Epilogue of the grouped kernels: combine the warps of the CTA per head, then either write
// the result (one split) or the split's partials; the last CTA of the (b, kvh) to arrive merges
// the splits of the group's heads (ticket on the group's first head, no waiting).  The ring
// is free by now and holds [warp][head][128] floats.
__device__ __forceinline__ void group_epilogue(const AttnParams& p, unsigned char* g_smem, int b, int head0, int gq,
                                               int split, float (&o)[16][4], float m0, float l0, float m1,
                                               float l1, float lt0, float lt1) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
  lt0 += __shfl_xor_sync(0xffffffffu, lt0, 1);
  lt0 += __shfl_xor_sync(0xffffffffu, lt0, 2);
  lt1 += __shfl_xor_sync(0xffffffffu, lt1, 1);
  lt1 += __shfl_xor_sync(0xffffffffu, lt1, 2);
  __syncthreads();
  float* sm_o = reinterpret_cast<float*>(g_smem);                       // 4 x 16 x 128 floats = 32 KB
  float* sm_m = sm_o + kTWarps * 16 * kHeadDim;                         // [warp][16]
  float* sm_l = sm_m + kTWarps * 16;
  float* sm_lt = sm_l + kTWarps * 16;
  __shared__ bool is_last;
#pragma unroll
  for (int nt = 0; nt < 16; ++nt) {
    *reinterpret_cast<float2*>(&sm_o[(warp * 16 + g) * kHeadDim + nt * 8 + 2 * tg]) = make_float2(o[nt][0], o[nt][1]);
    *reinterpret_cast<float2*>(&sm_o[(warp * 16 + g + 8) * kHeadDim + nt * 8 + 2 * tg]) = make_float2(o[nt][2], o[nt][3]);
  }
  if (tg == 0) {
    sm_m[warp * 16 + g] = m0; sm_l[warp * 16 + g] = l0; sm_lt[warp * 16 + g] = lt0;
    sm_m[warp * 16 + g + 8] = m1; sm_l[warp * 16 + g + 8] = l1; sm_lt[warp * 16 + g + 8] = lt1;
  }
  __syncthreads();
  auto finish = [&](int unit, float acc, float M, float L, float Lt) {
    p.out[(long long)unit * kHeadDim + tid] = __float2bfloat16_rn(Lt > 0.f ? acc / Lt : 0.f);
    if (tid == 0) {
      const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
      if (p.out_lse) p.out_lse[unit] = lse;
      if (p.out_delta) p.out_delta[unit] = L > 0.f ? -expm1f(lse - p.lse_full[unit]) : 1.f;
    }
  };
  for (int j = 0; j < gq; ++j) {
    const int unit = b * p.num_q_heads + head0 + j;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kTWarps; ++w) M = fmaxf(M, sm_m[w * 16 + j]);
    float acc = 0.f, L = 0.f, Lt = 0.f;
    if (M != -INFINITY) {
#pragma unroll
      for (int w = 0; w < kTWarps; ++w) {
        const float scw = exp2f(sm_m[w * 16 + j] - M);
        acc = fmaf(sm_o[(w * 16 + j) * kHeadDim + tid], scw, acc);
        L = fmaf(sm_l[w * 16 + j], scw, L);
        Lt = fmaf(sm_lt[w * 16 + j], scw, Lt);
      }
    }
    if (p.splits == 1) {
      finish(unit, acc, M, L, Lt);
    } else {
      float* part = p.partials + ((long long)unit * p.splits + split) * kPartStride;
      part[tid] = acc;
      if (tid == 0) { part[kHeadDim] = M; part[kHeadDim + 1] = L; part[kHeadDim + 2] = Lt; }
    }
  }
  if (p.splits == 1) return;
  __threadfence();
  __syncthreads();
  const int tunit = b * p.num_q_heads + head0;      // ticket slot: the group's first head
  if (tid == 0) {
    const unsigned int ticket = atomicAdd(p.tickets + tunit, 1u);
    is_last = (ticket == (unsigned int)p.splits - 1u);
    if (is_last) p.tickets[tunit] = 0u;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int j = 0; j < gq; ++j) {
    const int unit = tunit + j;
    const float* base = p.partials + (long long)unit * p.splits * kPartStride;
    float M = -INFINITY;
    for (int sp = 0; sp < p.splits; ++sp) M = fmaxf(M, __ldcg(base + sp * kPartStride + kHeadDim));
    float acc = 0.f, L = 0.f, Lt = 0.f;
    if (M != -INFINITY) {
      for (int sp = 0; sp < p.splits; ++sp) {
        const float scw = exp2f(__ldcg(base + sp * kPartStride + kHeadDim) - M);
        acc = fmaf(__ldcg(base + sp * kPartStride + tid), scw, acc);
        L = fmaf(__ldcg(base + sp * kPartStride + kHeadDim + 1), scw, L);
        Lt = fmaf(__ldcg(base + sp * kPartStride + kHeadDim + 2), scw, Lt);
      }
    }
    finish(unit, acc, M, L, Lt);
  }
}

__global__ void __launch_bounds__(kTThreads) dense_attn_mma_kernel(AttnParams p) {
  extern __shared__ __align__(128) unsigned char g_smem[];
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int gq = p.group_size;
  const int head0 = kvh * gq;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int t = __ldg(p.kv.seq_lens + b);
  int per = (t + p.splits * kTWarps - 1) / (p.splits * kTWarps);
  per = (per + kTStageRows - 1) & ~(kTStageRows - 1);
  const int start = min((split * kTWarps + warp) * per, t);
  const int end = min(start + per, t);
  const int nstages = (end - start + kTStageRows - 1) / kTStageRows;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(g_smem) + warp * (kTStages * kTStageBytes);
  const bool has0 = g < gq, has1 = g + 8 < gq;

  // A fragments of the group's queries: rows g and g + 8
  uint32_t aq[8][4];
  {
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + ((long long)b * p.num_q_heads + head0 + g) * kHeadDim);
    const uint32_t* q1 = q0 + 8 * (kHeadDim / 2);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      aq[ks][0] = has0 ? __ldg(q0 + ks * 8 + tg) : 0u;
      aq[ks][1] = has1 ? __ldg(q1 + ks * 8 + tg) : 0u;
      aq[ks][2] = has0 ? __ldg(q0 + ks * 8 + 4 + tg) : 0u;
      aq[ks][3] = has1 ? __ldg(q1 + ks * 8 + 4 + tg) : 0u;
    }
  }
  float o[16][4];
#pragma unroll
  for (int nt = 0; nt < 16; ++nt) { o[nt][0] = 0.f; o[nt][1] = 0.f; o[nt][2] = 0.f; o[nt][3] = 0.f; }
  float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;   // rows g and g + 8
  float lt0 = 0.f, lt1 = 0.f;

  const bool paged = p.kv.page_table != nullptr;
  const __nv_bfloat16* src_base = (lane < 16 ? p.kv.k : p.kv.v) + (lane & 15) * 8;
  const uint32_t dst_tile = (lane < 16 ? 0u : (uint32_t)kTTileBytes);
  const long long lin_off = (long long)b * p.kv.stride_outer + (long long)kvh * p.kv.stride_head;
  // paged: page id of the stage issued next, prefetched one stage ahead (start is a multiple of 16)
  auto page_of_stage = [&](int j) -> int {
    const int pos = start + j * kTStageRows;
    if (!paged || pos >= end) return 0;
    return __ldg(p.kv.page_table + (long long)b * p.kv.page_table_stride + (pos >> kPageShift));
  };
  int pg_next = page_of_stage(0);

  auto issue = [&](int j) {
    if (j < nstages) {
      const int pos0 = start + j * kTStageRows;
      long long row_off = lin_off + (long long)pos0 * kHeadDim;
      bool page_ok = true;
      if (paged) {
        const int page = pg_next;
        pg_next = page_of_stage(j + 1);
        page_ok = (unsigned)page < (unsigned)p.kv.num_pages;
        if (!page_ok) atomicOr(p.flags, kFlagBadPage);
        row_off = (long long)page * p.kv.stride_outer + (long long)kvh * p.kv.stride_head;
      }
      const uint32_t slot = ring + (uint32_t)(j % kTStages) * kTStageBytes + dst_tile;
#pragma unroll
      for (int r = 0; r < kTStageRows; ++r) {
        const bool ok = page_ok && (pos0 + r < end);
        const uint32_t dst = slot + r * kRowBytes + ((((uint32_t)lane & 15u) ^ (r & 7u)) << 4);
        cp_async_16(dst, src_base + (ok ? row_off + (long long)r * kHeadDim : 0ll), ok ? 16 : 0);
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int j = 0; j < kTStages - 1; ++j) issue(j);

  for (int i = 0; i < nstages; ++i) {
    cp_async_wait<kTStages - 2>();
    __syncwarp();
    issue(i + kTStages - 1);
    const uint32_t kt = ring + (uint32_t)(i % kTStages) * kTStageBytes;
    const int pos0 = start + i * kTStageRows;
    // keys of this lane: pos0 + 2tg, +1 (n-tile 0) and pos0 + 8 + 2tg, +1 (n-tile 1)
    group_stage(kt, kt + kTTileBytes, aq, pos0 + 2 * tg < end, pos0 + 2 * tg + 1 < end, pos0 + 8 + 2 * tg < end,
                pos0 + 9 + 2 * tg < end, o, m0, l0, m1, l1, lt0, lt1);
  }
  cp_async_wait<0>();
  group_epilogue(p, g_smem, b, head0, gq, split, o, m0, l0, m1, l1, lt0, lt1);
}

// ------------------------------------------------------- retrieval scoring, ring variant
// Logits a_i = q . k_i / sqrt(d) for all i < t (Eq. 2) with the K stream staged like the dense
// baseline's: warp-private cp.async ring (K tiles only, 6 stages of 16 rows), ldmatrix, one
// MMA tile for all heads of the KV group.  Writes fp32 logits [B][Hq][ld] and per-(head, split)
// online log-sum-exp partials part_ml[unit][split] in the log2 domain.
// grid (splits, Hkv, B).
constexpr int kSRStages = 6;
constexpr int kSRSmemBytes = kTWarps * kSRStages * kTTileBytes;      // 96 KB

struct ScoreParams {
  const __nv_bfloat16* q;
  KvDev kv;
  float* scores;          // [B][Hq][ld] or nullptr (log-sum-exp only)
  int ld;
  float2* part_ml;        // [B][Hq][splits]
  int splits, num_q_heads, group_size;
  const int* need;        // [B][Hq] or nullptr: score only KV heads with a query head that retrieves
  int group_max;          // 1: write max over the group's heads to the row of its first head only
  int chunk_rows;         // > 0: split j covers rows [j * chunk_rows, (j + 1) * chunk_rows) of every sequence
  uint32_t* flags;
};

// Group-shared ranking logits: the maximum over the heads on the tile rows (g and g + 8 of every
// lane quad) of the four logits a lane holds, stored by the lanes of row 0 into the row of the
// group's first head.  s[nt][2 hh + c]: n-tile nt, row half hh, column c.
template <int NT>
__device__ __forceinline__ void store_group_max(const float (&s)[NT][4], bool has0, bool has1, float* dst,
                                                int pos0, int end) {
  const int lane = threadIdx.x & 31;
  const int g = lane >> 2, tg = lane & 3;
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    float v[2];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      float x = fmaxf(has0 ? s[nt][c] : -INFINITY, has1 ? s[nt][2 + c] : -INFINITY);
      x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 4));
      x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 8));
      x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 16));
      v[c] = x * kScale;
    }
    const int key0 = pos0 + 8 * nt + 2 * tg;
    if (g == 0) {
      if (key0 + 1 < end) *reinterpret_cast<float2*>(dst + key0) = make_float2(v[0], v[1]);
      else if (key0 < end) dst[key0] = v[0];
    }
  }
}

__global__ void __launch_bounds__(kTThreads) score_ring_kernel(ScoreParams p) {
  extern __shared__ __align__(128) unsigned char g_smem[];
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int gq = p.group_size;
  const int head0 = kvh * gq;
  if (p.need != nullptr) {              // cosine-gated step: nothing to do if no head of the group retrieves
    bool any = false;
    for (int j = 0; j < gq; ++j) any |= __ldg(p.need + b * p.num_q_heads + head0 + j) != 0;
    if (!any) return;
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int t = __ldg(p.kv.seq_lens + b);
  int per = (t + p.splits * kTWarps - 1) / (p.splits * kTWarps);
  per = (per + kTStageRows - 1) & ~(kTStageRows - 1);
  const int start = min((split * kTWarps + warp) * per, t);
  const int end = min(start + per, t);
  const int nstages = (end - start + kTStageRows - 1) / kTStageRows;
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(g_smem) + warp * (kSRStages * kTTileBytes);
  const bool has0 = g < gq, has1 = g + 8 < gq;

  uint32_t aq[8][4];
  {
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + ((long long)b * p.num_q_heads + head0 + g) * kHeadDim);
    const uint32_t* q1 = q0 + 8 * (kHeadDim / 2);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      aq[ks][0] = has0 ? __ldg(q0 + ks * 8 + tg) : 0u;
      aq[ks][1] = has1 ? __ldg(q1 + ks * 8 + tg) : 0u;
      aq[ks][2] = has0 ? __ldg(q0 + ks * 8 + 4 + tg) : 0u;
      aq[ks][3] = has1 ? __ldg(q1 + ks * 8 + 4 + tg) : 0u;
    }
  }
  float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;

  const bool paged = p.kv.page_table != nullptr;
  // each lane copies 16 bytes; a K row is 16 lanes, so one instruction moves two rows
  const __nv_bfloat16* src_base = p.kv.k + (lane & 15) * 8;
  const int rsel = lane >> 4;                       // which of the two rows of a pair
  const long long lin_off = (long long)b * p.kv.stride_outer + (long long)kvh * p.kv.stride_head;
  auto page_of_stage = [&](int j) -> int {
    const int pos = start + j * kTStageRows;
    if (!paged || pos >= end) return 0;
    return __ldg(p.kv.page_table + (long long)b * p.kv.page_table_stride + (pos >> kPageShift));
  };
  int pg_next = page_of_stage(0);
  auto issue = [&](int j) {
    if (j < nstages) {
      const int pos0 = start + j * kTStageRows;
      long long row_off = lin_off + (long long)pos0 * kHeadDim;
      bool page_ok = true;
      if (paged) {
        const int page = pg_next;
        pg_next = page_of_stage(j + 1);
        page_ok = (unsigned)page < (unsigned)p.kv.num_pages;
        if (!page_ok) atomicOr(p.flags, kFlagBadPage);
        row_off = (long long)page * p.kv.stride_outer + (long long)kvh * p.kv.stride_head;
      }
      const uint32_t slot = ring + (uint32_t)(j % kSRStages) * kTTileBytes;
#pragma unroll
      for (int rp = 0; rp < kTStageRows / 2; ++rp) {
        const int r = 2 * rp + rsel;
        const bool ok = page_ok && (pos0 + r < end);
        const uint32_t dst = slot + r * kRowBytes + ((((uint32_t)lane & 15u) ^ (r & 7u)) << 4);
        cp_async_16(dst, src_base + (ok ? row_off + (long long)r * kHeadDim : 0ll), ok ? 16 : 0);
      }
    }
    cp_async_commit();
  };
#pragma unroll
  for (int j = 0; j < kSRStages - 1; ++j) issue(j);

  const int lm_mi = lane >> 3, lm_r = lane & 7;
  for (int i = 0; i < nstages; ++i) {
    cp_async_wait<kSRStages - 2>();
    __syncwarp();
    issue(i + kSRStages - 1);
    const uint32_t kt = ring + (uint32_t)(i % kSRStages) * kTTileBytes;
    const int pos0 = start + i * kTStageRows;
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
    for (int pp = 0; pp < 4; ++pp) {
      uint32_t bk0[4], bk1[4];
      ldmatrix_x4(bk0, kt + lm_r * kRowBytes + (((4 * pp + lm_mi) ^ (lm_r & 7)) << 4));
      ldmatrix_x4(bk1, kt + (8 + lm_r) * kRowBytes + (((4 * pp + lm_mi) ^ (lm_r & 7)) << 4));
      mma_bf16_full(s[0], aq[2 * pp][0], aq[2 * pp][1], aq[2 * pp][2], aq[2 * pp][3], bk0[0], bk0[1]);
      mma_bf16_full(s[1], aq[2 * pp][0], aq[2 * pp][1], aq[2 * pp][2], aq[2 * pp][3], bk1[0], bk1[1]);
      mma_bf16_full(s[0], aq[2 * pp + 1][0], aq[2 * pp + 1][1], aq[2 * pp + 1][2], aq[2 * pp + 1][3], bk0[2], bk0[3]);
      mma_bf16_full(s[1], aq[2 * pp + 1][0], aq[2 * pp + 1][1], aq[2 * pp + 1][2], aq[2 * pp + 1][3], bk1[2], bk1[3]);
    }
    // lane (g, tg): head g -> s[nt][0..1], head g + 8 -> s[nt][2..3]; keys pos0 + 8 nt + 2 tg, +1
    if (p.scores && p.group_max)
      store_group_max<2>(s, has0, has1, p.scores + ((long long)b * p.num_q_heads + head0) * p.ld, pos0, end);
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      if (hh == 0 ? has0 : has1) {
        float& m = hh == 0 ? m0 : m1;
        float& l = hh == 0 ? l0 : l1;
        float* dst = (p.scores && !p.group_max) ? p.scores + ((long long)b * p.num_q_heads + head0 + g + 8 * hh) * p.ld : nullptr;
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          const int key0 = pos0 + 8 * nt + 2 * tg;
          const float s0 = s[nt][2 * hh] * kScale, s1 = s[nt][2 * hh + 1] * kScale;
          if (key0 + 1 < end) {
            if (dst) *reinterpret_cast<float2*>(dst + key0) = make_float2(s0, s1);
            const float x0 = s0 * kLog2e, x1 = s1 * kLog2e;
            const float mn = fmaxf(m, fmaxf(x0, x1));
            l = l * exp2f(m - mn) + exp2f(x0 - mn) + exp2f(x1 - mn);
            m = mn;
          } else if (key0 < end) {
            if (dst) dst[key0] = s0;
            const float x0 = s0 * kLog2e;
            const float mn = fmaxf(m, x0);
            l = l * exp2f(m - mn) + exp2f(x0 - mn);
            m = mn;
          }
        }
      }
    }
  }
  cp_async_wait<0>();
  // ---- (m, l) per head: over the 4 lanes of a group, then over the warps
#pragma unroll
  for (int off = 1; off <= 2; off <<= 1) {
    float m2 = __shfl_xor_sync(0xffffffffu, m0, off), l2 = __shfl_xor_sync(0xffffffffu, l0, off);
    ml_combine(m0, l0, m2, l2);
    m2 = __shfl_xor_sync(0xffffffffu, m1, off);
    l2 = __shfl_xor_sync(0xffffffffu, l1, off);
    ml_combine(m1, l1, m2, l2);
  }
  __shared__ float sm_m[kTWarps][16], sm_l[kTWarps][16];
  if (tg == 0) {
    sm_m[warp][g] = m0; sm_l[warp][g] = l0;
    sm_m[warp][g + 8] = m1; sm_l[warp][g + 8] = l1;
  }
  __syncthreads();
  if (tid < gq) {
    float mm = -INFINITY, ll = 0.f;
    for (int w = 0; w < kTWarps; ++w) ml_combine(mm, ll, sm_m[w][tid], sm_l[w][tid]);
    p.part_ml[((long long)b * p.num_q_heads + head0 + tid) * p.splits + split] = make_float2(mm, ll);
  }
}

// ------------------------------------------------------------------- cosine gate (Eq. 9)
// One warp per (b, h).  `pos` = step % s is the position of this step in its block.  At
// pos == 0 the head retrieves into slot 0.  Later it shares the slot of the MOST RECENT earlier
// step of the block whose query has cosine similarity > tau with the current one, or, if
// there is none, retrieves into the next free slot (Sec. 4.1 "Similarity Criteria").
// Updates the block history (queries, slot per position, number of sets) and writes the
// decision: need (1 = retrieve now), slot (set to attend over), ref (position shared from, -1).
__global__ void __launch_bounds__(128)
gate_kernel(const __nv_bfloat16* __restrict__ q, int units, int pos, float tau, int slots,
            __nv_bfloat16* __restrict__ qhist, int* __restrict__ set_of_pos, int* __restrict__ nsets,
            int* __restrict__ need, int* __restrict__ slot_out, int* __restrict__ ref_out) {
  const int unit = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (unit >= units) return;
  const uint2 qx = *reinterpret_cast<const uint2*>(q + (long long)unit * kHeadDim + lane * 4);
  const float q0 = bf_lo(qx.x), q1 = bf_hi(qx.x), q2 = bf_lo(qx.y), q3 = bf_hi(qx.y);
  __nv_bfloat16* hist = qhist + (long long)unit * slots * kHeadDim;
  int ref = -1;
  if (pos > 0) {
    float qq = q0 * q0 + q1 * q1 + q2 * q2 + q3 * q3;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) qq += __shfl_xor_sync(0xffffffffu, qq, off);
    for (int j = pos - 1; j >= 0; --j) {
      const uint2 ex = *reinterpret_cast<const uint2*>(hist + (long long)j * kHeadDim + lane * 4);
      const float e0 = bf_lo(ex.x), e1 = bf_hi(ex.x), e2 = bf_lo(ex.y), e3 = bf_hi(ex.y);
      float dot = q0 * e0 + q1 * e1 + q2 * e2 + q3 * e3;
      float ee = e0 * e0 + e1 * e1 + e2 * e2 + e3 * e3;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) {
        dot += __shfl_xor_sync(0xffffffffu, dot, off);
        ee += __shfl_xor_sync(0xffffffffu, ee, off);
      }
      const float cs = dot / (sqrtf(qq) * sqrtf(ee));
      if (cs > tau) { ref = j; break; }      // uniform over the warp
    }
  }
  int slot;
  if (ref >= 0) {
    slot = set_of_pos[(long long)unit * slots + ref];
  } else {
    slot = pos == 0 ? 0 : min(nsets[unit], slots - 1);
  }
  *reinterpret_cast<uint2*>(hist + (long long)pos * kHeadDim + lane * 4) = qx;
  if (lane == 0) {
    if (ref < 0) nsets[unit] = slot + 1;
    set_of_pos[(long long)unit * slots + pos] = slot;
    need[unit] = ref < 0 ? 1 : 0;
    slot_out[unit] = slot;
    ref_out[unit] = ref;
  }
}

// Reduce the scoring pass' per-chunk (m, l) partials to lse_full (used when no selection runs).
__global__ void lse_reduce_kernel(const float2* __restrict__ part_ml, int nchunks, int chunk_rows,
                                  const int* __restrict__ seq_lens, int num_q_heads,
                                  float* __restrict__ lse_full, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const int t = __ldg(seq_lens + i / num_q_heads);
  // chunk_rows > 0: chunks past t were never written; 0: every partial is valid
  const int nch = chunk_rows > 0 ? min(nchunks, (t + chunk_rows - 1) / chunk_rows) : nchunks;
  float mm = -INFINITY, ll = 0.f;
  for (int c = 0; c < nch; ++c) {
    const float2 x = part_ml[(long long)i * nchunks + c];
    ml_combine(mm, ll, x.x, x.y);
  }
  lse_full[i] = ll > 0.f ? (mm + log2f(ll)) * kLn2 : -INFINITY;
}
// Diagnostic: is every unit's index list strictly ascending (hence unique), inside [0, t_b) and
// no longer than its stride?  One warp per (b, h); bad[unit] = 1 where it is not, *nbad counts.
__global__ void __launch_bounds__(128)
validate_lists_kernel(const int* __restrict__ idx, const int* __restrict__ count, int idx_stride,
                      const int* __restrict__ seq_lens, int num_q_heads, int units, int* bad, int* nbad) {
  const int unit = blockIdx.x * 4 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
  if (unit >= units) return;
  const int t = __ldg(seq_lens + unit / num_q_heads);
  const int n = __ldg(count + unit);
  const int* l = idx + (long long)unit * idx_stride;
  bool ok = n >= 0 && n <= idx_stride;
  const int m = min(max(n, 0), idx_stride);
  for (int i = lane; i < m; i += 32) {
    const int x = __ldg(l + i);
    if (x < 0 || x >= t) ok = false;
    if (i > 0 && __ldg(l + i - 1) >= x) ok = false;
  }
  ok = __all_sync(0xffffffffu, ok);
  if (lane == 0) {
    bad[unit] = ok ? 0 : 1;
    if (!ok) atomicAdd(nbad, 1);
  }
}

// One launch that takes a decode step's inputs straight from PINNED, device-mapped host memory:
// the queries into the staging buffer, the new K and V rows into the cache at position t_b - 1,
// the lengths into the device array.  Replaces four host-to-device copies and the append
// kernel: the transfers are 16-byte loads over the host link, all in flight at once.
// grid (batch, kIngestSplit), 256 threads.
constexpr int kIngestSplit = 4;
__global__ void __launch_bounds__(256)
ingest_kernel(const uint4* __restrict__ host_q, const uint4* __restrict__ host_k, const uint4* __restrict__ host_v,
              const int* __restrict__ host_lens, uint4* q_dev, __nv_bfloat16* k, __nv_bfloat16* v,
              long long stride_outer, long long stride_head, int* lens_dev, int hq, int hkv) {
  __shared__ int sh_t;
  const int b = blockIdx.x;
  if (threadIdx.x == 0) {
    sh_t = host_lens[b];
    if (blockIdx.y == 0) lens_dev[b] = sh_t;
  }
  __syncthreads();
  const int t = sh_t;
  const int nq = hq * 16, nk = hkv * 16;             // 16-byte items of this sequence
  const int total = nq + 2 * nk;
  for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < total; i += kIngestSplit * blockDim.x) {
    if (i < nq) {
      q_dev[(long long)b * nq + i] = host_q[(long long)b * nq + i];
    } else if (t > 0) {
      const int j = (i - nq) % nk, is_v = (i - nq) / nk;
      const int kvh = j >> 4, c = j & 15;
      const uint4 x = (is_v ? host_v : host_k)[(long long)b * nk + j];
      __nv_bfloat16* dst = (is_v ? v : k) + (long long)b * stride_outer + (long long)kvh * stride_head +
                           (long long)(t - 1) * kHeadDim + c * 8;
      *reinterpret_cast<uint4*>(dst) = x;
    }
  }
}


// Write the new token's K and V rows at position t_b - 1 (contiguous cache).
// grid (Hkv, B), 32 threads: lanes 0-15 copy the K row, lanes 16-31 the V row.
__global__ void append_rows_kernel(const __nv_bfloat16* __restrict__ new_k,
                                   const __nv_bfloat16* __restrict__ new_v, __nv_bfloat16* k,
                                   __nv_bfloat16* v, long long stride_outer, long long stride_head,
                                   const int* __restrict__ seq_lens, int num_kv_heads) {
  const int kvh = blockIdx.x, b = blockIdx.y;
  const int t = seq_lens[b];
  if (t <= 0) return;
  const int lane = threadIdx.x & 15;
  const long long src = ((long long)b * num_kv_heads + kvh) * kHeadDim + lane * 8;
  const long long dst = (long long)b * stride_outer + (long long)kvh * stride_head +
                        (long long)(t - 1) * kHeadDim + lane * 8;
  if (threadIdx.x < 16)
    *reinterpret_cast<uint4*>(k + dst) = *reinterpret_cast<const uint4*>(new_k + src);
  else
    *reinterpret_cast<uint4*>(v + dst) = *reinterpret_cast<const uint4*>(new_v + src);
}

}  // namespace prhs
