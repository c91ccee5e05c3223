// Gathered attention with the rows brought in by the TMA row gather (sm_100a).
//
// The arithmetic, the list handling and the row-id pipeline are those of gather_attn_mma_kernel;
// what changes is how a stage of 16 list entries reaches shared memory.  There every lane issued
// 16 cp.async copies per stage (one K row and one V row per instruction) and the ldmatrix / mma
// chain queued behind them; here 16 lanes issue ONE instruction together, each lane one
// `cp.async.bulk.tensor.2d.tile::gather4` that names four rows of K or of V by their row ids and
// one 64-column half of them, and the copy engine does the rest.  K and V are described as 2-D
// tensors [rows][128] bf16 with a box of one row by 64 columns and the 128-byte swizzle, so a
// stage lands as four [16 rows][64 columns] half tiles whose 16-byte chunks are XOR-swizzled by
// the row: ldmatrix reads them without bank conflicts, exactly as in the scoring kernel.
// Completion is an mbarrier per ring slot (expect_tx of the stage's 8 KB); every wait is bounded.
// Entries that are not real (past the end of the list, out of range) name a row beyond the
// tensor: the copy engine fills zeros there and the validity mask keeps them out of the softmax.
// No multicast.
//
// Selected by PRHS_CFG_TMA_GATHER only: it measured SLOWER than the cp.async kernel (a sharing
// step of the 32K-context layer at batch 8: 49.0 us against 44.1 us; the grouped-query stack at
// batch 16: 92 us against 72 us).  As a bare copy the row gather ties with cp.async when a row is
// one 256-byte box (44.0 us against 43.0 us), but a tile that ldmatrix can read without bank
// conflicts needs the 128-byte swizzle, whose boxes are at most 128 bytes wide: two boxes per row,
// twice the copy instructions, and at that granularity the copy engine is the bottleneck.
#pragma once
#include <cuda.h>

#include "attn.cuh"
#include "common.cuh"
#include "score_tma.cuh"

namespace prhs {

constexpr int kATStages = kTStages;                                  // 3 stages of 16 entries per warp
constexpr int kATHalfBytes = kTStageRows * 128;                      // one [16][64] bf16 half tile = 2 KB
constexpr int kATStageBytes = 4 * kATHalfBytes;                      // K half 0, K half 1, V half 0, V half 1
constexpr int kATSmemBytes = kTWarps * kATStages * kATStageBytes + 1024;   // + slack to align to 1 KB

__device__ __forceinline__ void tma_gather4_rows(uint32_t dst, const CUtensorMap* tm, int col, uint32_t r0, uint32_t r1,
                                                 uint32_t r2, uint32_t r3, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(tm), "r"(col), "r"((int)r0), "r"((int)r1), "r"((int)r2), "r"((int)r3), "r"(bar)
      : "memory");
}

// grid (splits, Hq, B), 128 threads.  tm_k / tm_v: K and V as [rows][128] bf16, box [1 row][64 columns],
// 128-byte swizzle; oob_row: a row coordinate outside the tensor.
__global__ void __launch_bounds__(kTThreads)
gather_attn_tma_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                       AttnParams p, uint32_t oob_row) {
  extern __shared__ unsigned char at_smem_raw[];
  __shared__ __align__(8) unsigned long long bars[kTWarps * kATStages];
  __shared__ int sh_abort;
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
  const uint32_t smem0 = ((uint32_t)__cvta_generic_to_shared(at_smem_raw) + 1023u) & ~1023u;
  const uint32_t ring = smem0 + warp * (kATStages * kATStageBytes);
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars) + 8 * warp * kATStages;

  if (tid == 0) sh_abort = 0;
  if (lane == 0) {
    for (int s = 0; s < kATStages; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

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
  // O^T += V^T P^T as in gather_attn_mma_kernel: eight 16 x 8 tiles whose column 0 is live
  float o[8][4];
#pragma unroll
  for (int mt = 0; mt < 8; ++mt) { o[mt][0] = 0.f; o[mt][1] = 0.f; o[mt][2] = 0.f; o[mt][3] = 0.f; }
  float m = -INFINITY, l = 0.f, lt = 0.f;

  // Row-id pipeline, 32 list entries (two stages) per step, one entry per lane (as in
  // gather_attn_mma_kernel): pos2 = raw list entry of group G + 2, pos1 / pg1 = checked position
  // and page id of group G + 1, rid_a = row id of group G, the one being issued.
  auto list_pos = [&](int grp) -> int { return list_entry(ld, start + grp * 32 + lane, end); };
  auto check_pos = [&](int pos, int grp) -> int {
    return checked_entry(ld, pos, start + grp * 32 + lane, end, t, p.flags);
  };
  const bool paged = p.kv.page_table != nullptr;
  auto page_of = [&](int pos) -> int {
    if (!paged || pos < 0) return 0;
    return __ldg(p.kv.page_table + (long long)b * p.kv.page_table_stride + (pos >> kPageShift));
  };
  auto row_id = [&](int pos, int page) -> uint32_t {
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
  uint32_t valid_a = __ballot_sync(0xffffffffu, rid_a != kBadRow);
  if (rid_a == kBadRow) rid_a = oob_row;       // the copy engine fills zeros for a row outside the tensor
  pos1 = check_pos(list_pos(1), 1);
  pg1 = page_of(pos1);
  int pos2 = list_pos(2);
  unsigned long long vmask = 0ull;     // 16 validity bits per ring slot

  // lanes 0-15 issue the stage's copies: lane = tensor (K, V) x column half x quad of rows
  const int my_quad = lane & 3, my_half = (lane >> 2) & 1, my_v = (lane >> 3) & 1;
  const uint32_t my_dst = (uint32_t)(my_v * 2 + my_half) * kATHalfBytes + (uint32_t)my_quad * 512u;
  const CUtensorMap* my_tm = my_v ? &tm_v : &tm_k;

  auto issue = [&](int j) {
    if (j >= nstages) return;
    if (j > 0 && (j & 1) == 0) {       // step the row-id pipeline
      const int grp = j >> 1;
      rid_a = row_id(pos1, pg1);
      valid_a = __ballot_sync(0xffffffffu, rid_a != kBadRow);
      if (rid_a == kBadRow) rid_a = oob_row;
      pos1 = check_pos(pos2, grp + 1);
      pg1 = page_of(pos1);
      pos2 = list_pos(grp + 2);
    }
    const int slot_i = j % kATStages;
    const uint32_t bar = bar0 + 8 * slot_i;
    const int src0 = (j & 1) * kTStageRows + 4 * my_quad;
    const uint32_t r0 = __shfl_sync(0xffffffffu, rid_a, src0), r1 = __shfl_sync(0xffffffffu, rid_a, src0 + 1);
    const uint32_t r2 = __shfl_sync(0xffffffffu, rid_a, src0 + 2), r3 = __shfl_sync(0xffffffffu, rid_a, src0 + 3);
    if (lane == 0) mbar_expect_tx(bar, kATStageBytes);
    __syncwarp();
    if (lane < 16)
      tma_gather4_rows(ring + (uint32_t)slot_i * kATStageBytes + my_dst, my_tm, 64 * my_half, r0, r1, r2, r3, bar);
    const uint32_t vm = (valid_a >> ((j & 1) * kTStageRows)) & 0xffffu;
    vmask = (vmask & ~(0xffffull << (16 * slot_i))) | ((unsigned long long)vm << (16 * slot_i));
  };

#pragma unroll
  for (int j = 0; j < kATStages - 1; ++j) issue(j);

  const float sc = kScale * kLog2e;
  const int lm_mi = lane >> 3, lm_r = lane & 7;
  const int vrow = (lm_mi & 1) * 8 + lm_r;
  for (int i = 0; i < nstages; ++i) {
    const int slot_i = i % kATStages;
    if (!__all_sync(0xffffffffu, mbar_wait(bar0 + 8 * slot_i, (i / kATStages) & 1, &sh_abort))) {
      if (lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
      break;
    }
    const uint32_t vm = (uint32_t)(vmask >> (16 * slot_i)) & 0xffffu;
    // the slot refilled now held stage i - 1, whose fragments the MMAs of the last iteration consumed
    issue(i + kATStages - 1);
    const uint32_t kt = ring + (uint32_t)slot_i * kATStageBytes;
    const uint32_t vt = kt + 2 * kATHalfBytes;
    // ---- S = Q K^T : all K fragments first, then the two accumulator chains interleaved
    uint32_t bk[2][4][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      const int row = nt * 8 + lm_r;
#pragma unroll
      for (int pp = 0; pp < 4; ++pp) {
        const int chunk = 4 * pp + lm_mi;          // 16-byte chunk of the 256-byte row
        ldmatrix_x4(bk[nt][pp], kt + (chunk >> 3) * kATHalfBytes + row * 128 + (((chunk & 7) ^ (row & 7)) << 4));
      }
    }
    float s[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
    float zq[2][2] = {{0.f, 0.f}, {0.f, 0.f}};      // dead accumulator rows, private to each chain
#pragma unroll
    for (int pp = 0; pp < 4; ++pp) {
      mma_bf16_row0(s[0][0], s[0][1], zq[0][0], zq[0][1], aq0[2 * pp], aq2[2 * pp], bk[0][pp][0], bk[0][pp][1]);
      mma_bf16_row0(s[1][0], s[1][1], zq[1][0], zq[1][1], aq0[2 * pp], aq2[2 * pp], bk[1][pp][0], bk[1][pp][1]);
      mma_bf16_row0(s[0][0], s[0][1], zq[0][0], zq[0][1], aq0[2 * pp + 1], aq2[2 * pp + 1], bk[0][pp][2], bk[0][pp][3]);
      mma_bf16_row0(s[1][0], s[1][1], zq[1][0], zq[1][1], aq0[2 * pp + 1], aq2[2 * pp + 1], bk[1][pp][2], bk[1][pp][3]);
    }
    // the first half of the V fragments, fetched under the softmax arithmetic
    auto v_addr = [&](int np) -> uint32_t {
      const int chunk = 2 * np + (lm_mi >> 1);
      return vt + (chunk >> 3) * kATHalfBytes + vrow * 128 + (((chunk & 7) ^ (vrow & 7)) << 4);
    };
    uint32_t bv[4][4];
#pragma unroll
    for (int np = 0; np < 4; ++np) ldmatrix_x4_trans(bv[np], v_addr(np));
    // ---- online softmax on the 16 logits held by lanes 0-3 (lazy reference exponent)
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
      // ---- O^T += V^T P^T
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) mma_bf16_full(o[mt], bv[mt][0], bv[mt][2], bv[mt][1], bv[mt][3], ap0, ap2);
#pragma unroll
      for (int np = 4; np < 8; ++np) ldmatrix_x4_trans(bv[np - 4], v_addr(np));
#pragma unroll
      for (int mt = 4; mt < 8; ++mt)
        mma_bf16_full(o[mt], bv[mt - 4][0], bv[mt - 4][2], bv[mt - 4][1], bv[mt - 4][3], ap0, ap2);
    }
  }
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
  // after an aborted wait copies may still be in flight towards this CTA's shared memory: one
  // more bounded wait per barrier of the warp before anybody returns
  if (sh_abort && lane == 0) {
    for (int s = 0; s < kATStages; ++s) {
      const long long t0 = clock64();
      while (!mbar_try_wait(bar0 + 8 * s, 0) && !mbar_try_wait(bar0 + 8 * s, 1))
        if (clock64() - t0 > kWaitBudgetCycles / 8) break;
    }
  }
  if (sh_abort) __syncthreads();
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

}  // namespace prhs
