// Gathered attention with ONE index set per (sequence, KV head), shared by the query heads of
// the group (a labelled variant for grouped-query attention; the paper's sets are per head,
// Sec. 4.1).  A gathered K/V row is fetched once and serves every head of the group: the heads
// sit on the rows of the MMA tile as in the dense baseline (head j of the group = row j), the
// rows arrive through the warp-private cp.async ring and the staged row-id pipeline of the
// per-head gathered kernel, and the list is generated in the kernel from (S0, M, W).
// grid (splits, Hkv, B).  Partials, tickets, outputs and delta are per query head.
#pragma once
#include "attn.cuh"

namespace prhs {

__global__ void __launch_bounds__(kTThreads) gather_group_attn_mma_kernel(AttnParams p) {
  extern __shared__ __align__(128) unsigned char g_smem[];
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int gq = p.group_size;
  const int head0 = kvh * gq;
  const int unit0 = b * p.num_q_heads + head0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const int t = __ldg(p.kv.seq_lens + b);
  const ListDesc ld = make_list_desc(p, unit0, t);
  const int cnt = ld.count;
  int per = (cnt + p.splits * kTWarps - 1) / (p.splits * kTWarps);
  per = (per + kTStageRows - 1) & ~(kTStageRows - 1);
  const int start = min((split * kTWarps + warp) * per, cnt);
  const int end = min(start + per, cnt);
  const int nstages = (end - start + kTStageRows - 1) / kTStageRows;
  const uint32_t outer_rows = (uint32_t)(p.kv.stride_outer >> 7);
  const uint32_t head_rows = (uint32_t)(p.kv.stride_head >> 7);
  const uint32_t ring = (uint32_t)__cvta_generic_to_shared(g_smem) + warp * (kTStages * kTStageBytes);
  const bool has0 = g < gq, has1 = g + 8 < gq;

  // A fragments of the group's queries: rows g and g + 8
  uint32_t aq[8][4];
  {
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + ((long long)unit0 + g) * kHeadDim);
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
  float lt0 = 0.f, lt1 = 0.f;                                 // sums of the weights as rounded to bf16

  // Row-id pipeline, 32 list entries (two stages) per step, one entry per lane; every level is
  // produced one step before it is consumed (see gather_attn_mma_kernel).
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
  if (rid_a == kBadRow) rid_a = 0u;
  pos1 = check_pos(list_pos(1), 1);
  pg1 = page_of(pos1);
  int pos2 = list_pos(2);

  // the copy of a row as in gather_attn_mma_kernel: lane p fills position p with source chunk p ^ (r & 7)
  const __nv_bfloat16* srcx[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) srcx[k] = (lane < 16 ? p.kv.k : p.kv.v) + ((((uint32_t)lane & 15u) ^ (uint32_t)k) << 3);
  const uint32_t dst_lane = (lane < 16 ? 0u : (uint32_t)kTTileBytes) + (((uint32_t)lane & 15u) << 4);
  uint32_t vmv[kTStages];              // 16 validity bits per ring slot
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

  auto stage = [&](int i, auto slot_c) {
    constexpr int kSlot = decltype(slot_c)::value;
    cp_async_wait<kTStages - 2>();
    __syncwarp();
    const uint32_t vm = vmv[kSlot];
    issue(i + kTStages - 1, SlotC<(kSlot + kTStages - 1) % kTStages>{});
    const uint32_t kt = ring + (uint32_t)kSlot * kTStageBytes;
    group_stage(kt, kt + kTTileBytes, aq, (vm >> (2 * tg)) & 1u, (vm >> (2 * tg + 1)) & 1u,
                (vm >> (8 + 2 * tg)) & 1u, (vm >> (9 + 2 * tg)) & 1u, o, m0, l0, m1, l1, lt0, lt1);
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
  group_epilogue(p, g_smem, b, head0, gq, split, o, m0, l0, m1, l1, lt0, lt1);
}

}  // namespace prhs
