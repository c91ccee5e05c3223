// Gathered attention with one index set per (sequence, KV head) (the labelled grouped-query
// variant of attn_group.cuh) on the tcgen05 tensor cores.
//
// One CTA per (split, KV head, sequence) walks its slice of the list in tiles of 128 rows:
//   * two sets of four loader warps take the even and the odd tiles: a warp gathers 32 of the tile's
//     K rows and V rows (256 bytes each, 16-byte cp.async, zero fill for entries that are masked),
//     waits for them, and signals; while one set waits for its tile to land the other issues the
//     next.  Every row is written in the 128-byte-swizzled layout the tensor core reads through a
//     matrix descriptor: a K tile is K-major for S = K Q^T, and the same physical layout of a V
//     tile is MN-major for O^T = V^T P^T (the 128 dimensions are the M rows there).  K tiles live
//     in a ring of two, one per set (a K tile is free as soon as its S has been computed), V tiles
//     in a ring of four (a V tile waits for the softmax of its tile);
//   * one thread issues S[128 keys x 16 heads] = K_j Q^T into one of two accumulators in tensor
//     memory, another O_a^T[128 dims x 16 heads] += V_j^T P_j^T;
//   * two groups of four softmax warps take the even and the odd tiles.  A thread owns one key of
//     its group's tiles (a lane of tensor memory): it reads the key's logits for the group's heads,
//     writes the bf16 weights into its group's 16 x 128 P tile (K-major, swizzled) and keeps the
//     sums.  Each group has its own O accumulator and running maxima, like two splits of the list
//     inside the CTA; they are merged at the end.  A group raises its running maximum -- and
//     rescales its O in tensor memory -- only when some logit exceeds it by more than 2^8: a vote
//     per tile (one named barrier), the maximum reduction only when the vote says so.
// No register accumulators (the mma.sync kernel holds 64 per thread), no ldmatrix.  Partials, tickets,
// outputs and delta are per query head, as in the mma.sync kernel.  Every mbarrier wait is bounded;
// tensor memory is freed on every path.
//
// The kernel is a template over the shape of a CTA (GUShape below): two softmax groups and two loader sets
// as described (18 warps, a 205 KB ring, one CTA per SM), or one of each (10 warps, 109 KB, two CTAs per
// SM); the library launches the second where there are more units than SMs.
//
// Selected by PRHS_CFG_GROUP_TCGEN05 only.  Measured against the mma.sync kernel (sharing step of the
// group-shared variant, us): 32K contexts at batch 16: 44.5 against 42.6; 128K at batch 4: 40.3 against
// 34.3; the ragged paged batch of 64: 128 against 120.  With one CTA per SM the per-CTA set-up and merge
// (about 7 us: list description, tensor-memory allocation, Q tile; partials, ticket) is not covered by a
// second CTA as it is for the mma.sync kernel; with two per SM each has room for one K tile and two V
// tiles only, and a tile passes through four agents (loader set, S issue, softmax group, O issue), so a
// stage stays occupied for about 3 us.  Other arrangements measured slower (three loader sets with three
// K and three V stages: 52.6 us at the first shape; two sets with three and three: 46.5).
#pragma once
#include "attn.cuh"
#include "score_umma.cuh"

namespace prhs {

constexpr int kGUTileRows = 128;
constexpr int kGUHalfBytes = kGUTileRows * 128;          // [128 rows][64 columns] bf16
constexpr int kGUTileBytes = 2 * kGUHalfBytes;           // one K or V tile: 32 KB
constexpr int kGUQBytes = 2 * kSUHeads * 128;            // Q tile, and each of the two P tiles: 4 KB
// Shape of a CTA: G softmax groups (1 or 2), SETS loader sets (1 or 2); K stages = SETS (one per set), V
// stages = 2 SETS.  (2, 2): 18 warps and a 205 KB ring, one CTA per SM.  (1, 1): 10 warps and 109 KB, two CTAs
// per SM, each with a shallower pipeline, covering each other's set-up and merge.
template <int G, int SETS>
struct GUShape {
  static constexpr int kKStages = SETS, kVStages = 2 * SETS;
  static constexpr int kLoaderWarp0 = 4 * G, kQKWarp = 4 * G + 4 * SETS, kPVWarp = kQKWarp + 1;
  static constexpr int kThreads = (kPVWarp + 1) * 32;
  static constexpr int kSmemBytes = (kKStages + kVStages) * kGUTileBytes + 3 * kGUQBytes + 1024;
  static constexpr int kCtasPerSm = (G == 1 && SETS == 1) ? 2 : 1;
};
constexpr int kGUTmemCols = 64;                          // S0, S1, O0, O1: 16 fp32 columns each
constexpr uint32_t kGUIdescQK = kSUIdesc;                // A = K tile (K-major), B = Q tile (K-major)
constexpr uint32_t kGUIdescPV = kSUIdesc | (1u << 15);   // A = V tile read MN-major, B = P tile (K-major)
constexpr float kGURescaleGap = 8.f;                     // log2 units a logit may exceed the running maximum

// V tile as the MN-major A operand: 64-dimension blocks 16 KB apart (leading offset), groups of
// eight key rows 1024 bytes apart (stride offset), 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc_mn(uint32_t smem_addr) {
  return ((uint64_t)kSUDescHi << 32) | (uint64_t)(((smem_addr >> 4) & 0x3fffu) | ((uint32_t)(kGUHalfBytes >> 4) << 16));
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
        "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15]))
      : "memory");
  asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
// named barriers: 1 and 2 = the softmax groups (128 threads each), 3 = both groups
__device__ __forceinline__ void group_bar(int g) { asm volatile("bar.sync %0, 128;" ::"r"(g + 1) : "memory"); }
__device__ __forceinline__ void groups_bar() { asm volatile("bar.sync 3, 256;" ::: "memory"); }   // G = 2 only

// grid (splits, Hkv, B), GUShape<G, SETS>::kThreads threads.
template <int G, int SETS>
__global__ void __launch_bounds__(GUShape<G, SETS>::kThreads, GUShape<G, SETS>::kCtasPerSm)
gather_group_attn_umma_kernel(AttnParams p) {
  using Shape = GUShape<G, SETS>;
  constexpr int kGUKStages = Shape::kKStages, kGUVStages = Shape::kVStages, kGUThreads = Shape::kThreads;
  extern __shared__ unsigned char gu_smem_raw[];
  // full[0..4), k_empty[4..6), v_empty[6..10), s_full[10..12), s_empty[12..14), p_full[14..16), p_empty[16..18),
  // o_done[18], drain[19..21).  A wait names a phase by its parity, which is only sound for a waiter that
  // follows the barrier phase by phase: every barrier here is waited for, use after use, by the same agent.
  __shared__ __align__(8) unsigned long long bars[21];
  __shared__ uint32_t vmask[kGUVStages][4];
  __shared__ int exceed_flag[2][3];
  __shared__ float red_max[2][4][kSUHeads];
  __shared__ float red_l[2][4][kSUHeads], red_lt[2][4][kSUHeads];
  __shared__ float other_m[kSUHeads];
  __shared__ uint32_t tmem_slot;
  __shared__ int sh_abort;
  __shared__ bool is_last;
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int gq = p.group_size;
  const int head0 = kvh * gq;
  const int unit0 = b * p.num_q_heads + head0;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = __ldg(p.kv.seq_lens + b);
  const ListDesc ld = make_list_desc(p, unit0, t);
  const int cnt = ld.count;
  int per = (cnt + p.splits - 1) / p.splits;
  per = (per + kGUTileRows - 1) & ~(kGUTileRows - 1);
  const int start = min(split * per, cnt);
  const int end = min(start + per, cnt);
  const int ntiles = (end - start + kGUTileRows - 1) / kGUTileRows;
  const uint32_t smem0 = ((uint32_t)__cvta_generic_to_shared(gu_smem_raw) + 1023u) & ~1023u;
  const uint32_t v_ring = smem0 + kGUKStages * kGUTileBytes;
  const uint32_t q_smem = v_ring + kGUVStages * kGUTileBytes;
  const uint32_t p_smem = q_smem + kGUQBytes;            // two P tiles
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  const uint32_t bar_full = bar0, bar_kempty = bar0 + 8 * 4, bar_vempty = bar0 + 8 * 6, bar_sfull = bar0 + 8 * 10;
  const uint32_t bar_sempty = bar0 + 8 * 12, bar_pfull = bar0 + 8 * 14, bar_pempty = bar0 + 8 * 16;
  const uint32_t bar_odone = bar0 + 8 * 18, bar_drain = bar0 + 8 * 19;

  if (tid == 0) {
    for (int s = 0; s < kGUVStages; ++s) {
      mbar_init(bar_full + 8 * s, 4);      // one arrive per warp of the loader set that brought the tile
      mbar_init(bar_vempty + 8 * s, 1);    // a commit of the PV thread
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_kempty + 8 * a, 1);    // a commit of the QK thread
      mbar_init(bar_sfull + 8 * a, 1);     // a commit of the QK thread
      mbar_init(bar_sempty + 8 * a, 4);    // one arrive per softmax warp of the group
      mbar_init(bar_pfull + 8 * a, 4);     // one arrive per softmax warp of the group
      mbar_init(bar_pempty + 8 * a, 1);    // a commit of the PV thread
      mbar_init(bar_drain + 8 * a, 1);
      for (int i = 0; i < 3; ++i) exceed_flag[a][i] = 0;
    }
    mbar_init(bar_odone, 1);
    sh_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Q tile (rows of absent heads zero) and the two P tiles (zero)
  for (int i = tid; i < 3 * kSUHeads * 16; i += kGUThreads) {
    const int tile = i / (kSUHeads * 16), r = i % (kSUHeads * 16);
    const int h = r >> 4, c16 = r & 15, hf = c16 >> 3, c = c16 & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (tile == 0 && h < gq) v = __ldg(reinterpret_cast<const uint4*>(p.q + ((long long)unit0 + h) * kHeadDim) + c16);
    const uint32_t dst = q_smem + tile * kGUQBytes + hf * (kSUHeads * 128) + h * 128 + ((c ^ (h & 7)) << 4);
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == Shape::kQKWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(&tmem_slot)), "r"((uint32_t)kGUTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem0 = *(volatile uint32_t*)&tmem_slot;

  if (warp < Shape::kLoaderWarp0) {
    // ---------------- softmax groups: group g takes the tiles j = g, g + 2, ...; a thread is key
    // row `row` of each of them, and dimension `row` of the group's O^T
    const int g = G == 2 ? warp >> 2 : 0;
    const int row = tid & 127;
    const uint32_t lane_base = (uint32_t)(32 * (warp & 3)) << 16;
    const uint32_t tmem_o = tmem0 + (uint32_t)((2 + g) * kSUHeads) + lane_base;
    float m_run[kSUHeads], l_run[kSUHeads], lt_run[kSUHeads];
#pragma unroll
    for (int h = 0; h < kSUHeads; ++h) { m_run[h] = -INFINITY; l_run[h] = 0.f; lt_run[h] = 0.f; }
    // A warp whose wait runs out sets `aborted` and keeps looping without touching anything, so that
    // the four warps of a group execute the same number of named barriers whatever happens.
    bool aborted = false;
    for (int j = g, i = 0; j < ntiles; j += G, ++i) {
      const int stage = j % kGUVStages;
      const int a = j & 1, ua = j >> 1;          // S and P buffer of the tile, and which use of them this is
      const uint32_t tmem_s = tmem0 + (uint32_t)(a * kSUHeads) + lane_base;
      float s[16];
      bool exceed = false;
      if (!aborted) {
        bool ok = mbar_wait(bar_sfull + 8 * a, ua & 1, &sh_abort);
        if (ok) ok = mbar_wait(bar_full + 8 * stage, (j / kGUVStages) & 1, &sh_abort);
        aborted = !__all_sync(0xffffffffu, ok);
      }
      if (!aborted) {
        tc_fence_after();
        tmem_ld16(tmem_s, s);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_sempty + 8 * a);
        const bool valid = ((vmask[stage][warp & 3] >> lane) & 1u) != 0u && start + j * kGUTileRows + row < end;
        // logits in the log2 domain; does any exceed its head's running maximum by more than the gap?
#pragma unroll
        for (int h = 0; h < kSUHeads; ++h) {
          if (h < gq) {
            s[h] = valid ? s[h] * (kScale * kLog2e) : -INFINITY;
            exceed = exceed || s[h] > m_run[h] + kGURescaleGap;
          }
        }
        exceed = __any_sync(0xffffffffu, exceed);
        if (lane == 0 && exceed) exceed_flag[g][i % 3] = 1;
      }
      if (row == 0) exceed_flag[g][(i + 1) % 3] = 0;      // the next tile's flag (last read two barriers ago)
      group_bar(g);
      const bool raise = !aborted && exceed_flag[g][i % 3] != 0;
      const bool any_raise = exceed_flag[g][i % 3] != 0;   // the same for every thread of the group
      float fac[kSUHeads];
#pragma unroll
      for (int h = 0; h < kSUHeads; ++h) fac[h] = 1.f;
      if (any_raise) {
        // the tile's maximum per head over its 128 keys, then the new running maxima
        if (!aborted) {
#pragma unroll
          for (int h = 0; h < kSUHeads; ++h) {
            if (h < gq) {
              float v = s[h];
#pragma unroll
              for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
              if (lane == 0) red_max[g][warp & 3][h] = v;
            }
          }
        }
        group_bar(g);
        if (raise) {
#pragma unroll
          for (int h = 0; h < kSUHeads; ++h) {
            if (h < gq) {
              const float mt = fmaxf(fmaxf(red_max[g][0][h], red_max[g][1][h]), fmaxf(red_max[g][2][h], red_max[g][3][h]));
              if (mt > m_run[h] + kGURescaleGap) {         // also the first finite maximum (m_run = -inf)
                fac[h] = exp2f(m_run[h] - mt);             // 0 while nothing has been accumulated
                l_run[h] *= fac[h];
                lt_run[h] *= fac[h];
                m_run[h] = mt;
              }
            }
          }
        }
        group_bar(g);                                      // red_max may be rewritten by the next raise
      }
      if (aborted) continue;
      // the P buffer's previous tile has been consumed; with two groups that is the group's previous tile,
      // whose MMAs into O have then landed too; a single group asks for its previous tile's separately
      if (ua >= 1 && !__all_sync(0xffffffffu, mbar_wait(bar_pempty + 8 * a, (ua - 1) & 1, &sh_abort))) {
        aborted = true;
        continue;
      }
      if (G == 1 && raise && j >= 1 &&
          !__all_sync(0xffffffffu, mbar_wait(bar_pempty + 8 * (a ^ 1), ((j - 1) >> 1) & 1, &sh_abort))) {
        aborted = true;
        continue;
      }
      if (raise && i >= 1) {
        // O of the group's tiles so far, scaled to the new maxima; the MMAs of this tile are not issued
        // before this warp's arrive on p_full below
        tc_fence_after();
        float o[16];
        tmem_ld16(tmem_o, o);
#pragma unroll
        for (int h = 0; h < kSUHeads; ++h) o[h] *= fac[h];
        tmem_st16(tmem_o, o);
        tc_fence_before();
      }
      const uint32_t pdst = p_smem + a * kGUQBytes + (row >> 6) * (kSUHeads * 128) + (row & 7) * 2;
      const int pc = (row & 63) >> 3;
#pragma unroll
      for (int h = 0; h < kSUHeads; ++h) {
        if (h < gq) {
          const float pv = (s[h] > -INFINITY) ? exp2f(s[h] - m_run[h]) : 0.f;
          const __nv_bfloat16 pb = __float2bfloat16_rn(pv);
          l_run[h] += pv;
          lt_run[h] += __bfloat162float(pb);
          asm volatile("st.shared.b16 [%0], %1;" ::"r"(pdst + h * 128 + ((pc ^ (h & 7)) << 4)), "h"(__bfloat16_as_ushort(pb)) : "memory");
        }
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_pfull + 8 * a);
    }
    if (aborted && lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
    // ---- the group's result: O^T[row][head], the sums over its keys
    float o[16];
#pragma unroll
    for (int h = 0; h < kSUHeads; ++h) o[h] = 0.f;
    // both groups wait for the last MMA (also the one without tiles: it writes into the ring below)
    bool have_o = !aborted && ntiles > 0;
    if (have_o) {
      have_o = __all_sync(0xffffffffu, mbar_wait(bar_odone, 0, &sh_abort));
      if (!have_o && lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
    }
    if (have_o && ntiles > g) {
      tc_fence_after();
      tmem_ld16(tmem_o, o);
      tc_fence_before();
    }
#pragma unroll
    for (int h = 0; h < kSUHeads; ++h) {
      if (h < gq) {
        float l = l_run[h], lt = lt_run[h];
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
          l += __shfl_xor_sync(0xffffffffu, l, off);
          lt += __shfl_xor_sync(0xffffffffu, lt, off);
        }
        if (lane == 0) { red_l[g][warp & 3][h] = l; red_lt[g][warp & 3][h] = lt; }
      }
    }
    // ---- the odd tiles' group hands its result to the even tiles' group through the (free) ring
    float* xo = reinterpret_cast<float*>(gu_smem_raw + (smem0 - (uint32_t)__cvta_generic_to_shared(gu_smem_raw)));
    if (G == 2 && g == 1) {
#pragma unroll
      for (int h = 0; h < kSUHeads; ++h)
        if (h < gq) xo[h * kGUTileRows + row] = o[h];
      if (row == 0) {
#pragma unroll
        for (int h = 0; h < kSUHeads; ++h)
          if (h < gq) other_m[h] = m_run[h];
      }
    }
    if (G == 2) groups_bar();
    else group_bar(0);
    if (g == 0) {
      float M[kSUHeads], L[kSUHeads], Lt[kSUHeads];
#pragma unroll
      for (int h = 0; h < kSUHeads; ++h) {
        if (h < gq) {
          const float l0 = red_l[0][0][h] + red_l[0][1][h] + red_l[0][2][h] + red_l[0][3][h];
          const float t0 = red_lt[0][0][h] + red_lt[0][1][h] + red_lt[0][2][h] + red_lt[0][3][h];
          const float l1 = G == 2 ? red_l[1][0][h] + red_l[1][1][h] + red_l[1][2][h] + red_l[1][3][h] : 0.f;
          const float t1 = G == 2 ? red_lt[1][0][h] + red_lt[1][1][h] + red_lt[1][2][h] + red_lt[1][3][h] : 0.f;
          const float m1 = G == 2 ? other_m[h] : -INFINITY;
          const float mm = fmaxf(m_run[h], m1);
          const float f0 = mm > -INFINITY ? exp2f(m_run[h] - mm) : 0.f, f1 = mm > -INFINITY ? exp2f(m1 - mm) : 0.f;
          M[h] = mm;
          L[h] = l0 * f0 + l1 * f1;
          Lt[h] = t0 * f0 + t1 * f1;
          o[h] = o[h] * f0 + (G == 2 ? xo[h * kGUTileRows + row] * f1 : 0.f);
        }
      }
      auto finish = [&](int unit, float acc, float Mx, float Lx, float Ltx) {
        p.out[(long long)unit * kHeadDim + row] = __float2bfloat16_rn(Ltx > 0.f ? acc / Ltx : 0.f);
        if (row == 0) {
          const float lse = Lx > 0.f ? (Mx + log2f(Lx)) * kLn2 : -INFINITY;
          if (p.out_lse) p.out_lse[unit] = lse;
          if (p.out_delta) p.out_delta[unit] = Lx > 0.f ? -expm1f(lse - p.lse_full[unit]) : 1.f;
        }
      };
#pragma unroll
      for (int h = 0; h < kSUHeads; ++h) {
        if (h < gq) {
          const int unit = unit0 + h;
          if (p.splits == 1) {
            finish(unit, o[h], M[h], L[h], Lt[h]);
          } else {
            float* part = p.partials + ((long long)unit * p.splits + split) * kPartStride;
            part[row] = o[h];
            if (row == 0) { part[kHeadDim] = M[h]; part[kHeadDim + 1] = L[h]; part[kHeadDim + 2] = Lt[h]; }
          }
        }
      }
      if (p.splits > 1) {
        __threadfence();
        group_bar(0);
        if (row == 0) {
          const unsigned int ticket = atomicAdd(p.tickets + unit0, 1u);
          is_last = (ticket == (unsigned int)p.splits - 1u);
          if (is_last) p.tickets[unit0] = 0u;
        }
        group_bar(0);
        if (is_last) {
          __threadfence();
          for (int h = 0; h < gq; ++h) {
            const int unit = unit0 + h;
            const float* base = p.partials + (long long)unit * p.splits * kPartStride;
            float Mx = -INFINITY;
            for (int sp = 0; sp < p.splits; ++sp) Mx = fmaxf(Mx, __ldcg(base + sp * kPartStride + kHeadDim));
            float acc = 0.f, Lx = 0.f, Ltx = 0.f;
            if (Mx != -INFINITY) {
              for (int sp = 0; sp < p.splits; ++sp) {
                const float scw = exp2f(__ldcg(base + sp * kPartStride + kHeadDim) - Mx);
                acc = fmaf(__ldcg(base + sp * kPartStride + row), scw, acc);
                Lx = fmaf(__ldcg(base + sp * kPartStride + kHeadDim + 1), scw, Lx);
                Ltx = fmaf(__ldcg(base + sp * kPartStride + kHeadDim + 2), scw, Ltx);
              }
            }
            finish(unit, acc, Mx, Lx, Ltx);
          }
        }
      }
    }
  } else if (warp < Shape::kQKWarp) {
    // ---------------- loader warps: set ls brings the tiles j = ls, ls + SETS, ... (K stage ls, V stage j mod 2 SETS),
    // warp `band` of the set the rows 32 band .. + 31 of each; lanes 0-15 copy a K row, lanes 16-31 the V
    // row of the same entry
    const int ls = (warp - Shape::kLoaderWarp0) >> 2, band = (warp - Shape::kLoaderWarp0) & 3;
    const bool paged = p.kv.page_table != nullptr;
    const uint32_t outer_rows = (uint32_t)(p.kv.stride_outer >> 7), head_rows = (uint32_t)(p.kv.stride_head >> 7);
    const int c = lane & 15;
    const __nv_bfloat16* src = (lane < 16 ? p.kv.k : p.kv.v) + c * 8;
    const uint32_t dst_lane = (uint32_t)(c >> 3) * kGUHalfBytes;
    const int jl0 = start + band * 32 + lane;
    int pos_next = list_entry(ld, jl0 + ls * kGUTileRows, end);
    // row id of this lane's entry of tile j (0 and a cleared bit of vm if it is masked); also starts the load
    // of the entry of the set's next tile
    auto lookup = [&](int j, uint32_t& rid, uint32_t& vm) {
      const int jl = jl0 + j * kGUTileRows;
      const int pos = checked_entry(ld, pos_next, jl, end, t, p.flags);
      if (j + SETS < ntiles) pos_next = list_entry(ld, jl + SETS * kGUTileRows, end);
      rid = kBadRow;
      if (pos >= 0) {
        if (paged) {
          const int page = __ldg(p.kv.page_table + (long long)b * p.kv.page_table_stride + (pos >> kPageShift));
          if ((unsigned)page >= (unsigned)p.kv.num_pages) atomicOr(p.flags, kFlagBadPage);
          else rid = (uint32_t)page * outer_rows + (uint32_t)kvh * head_rows + (uint32_t)(pos & 15);
        } else {
          rid = (uint32_t)b * outer_rows + (uint32_t)kvh * head_rows + (uint32_t)pos;
        }
      }
      vm = __ballot_sync(0xffffffffu, rid != kBadRow);
      if (rid == kBadRow) rid = 0u;
    };
    uint32_t rid = 0u, vm = 0u;
    if (ls < ntiles) lookup(ls, rid, vm);
    bool aborted = false;
    for (int j = ls, i = 0; j < ntiles; j += SETS, ++i) {
      const int stage = j % kGUVStages;
      // the set's K stage was last read by the S of the set's previous tile, the V stage by the O of the one before
      bool ok = true;
      if (i >= 1) ok = mbar_wait(bar_kempty + 8 * ls, (i - 1) & 1, &sh_abort);
      if (ok && j >= kGUVStages) ok = mbar_wait(bar_vempty + 8 * stage, ((j / kGUVStages) - 1) & 1, &sh_abort);
      if (!__all_sync(0xffffffffu, ok)) {
        aborted = true;
        break;
      }
      if (lane == 0) vmask[stage][band] = vm;
      const uint32_t tile = (lane < 16 ? smem0 + (uint32_t)ls * kGUTileBytes : v_ring + (uint32_t)stage * kGUTileBytes) + dst_lane;
#pragma unroll 8
      for (int r = 0; r < 32; ++r) {
        const uint32_t rr = __shfl_sync(0xffffffffu, rid, r);
        const int trow = band * 32 + r;
        cp_async_16(tile + trow * 128 + (((c & 7) ^ (trow & 7)) << 4), src + (size_t)rr * kHeadDim, ((vm >> r) & 1u) ? 16 : 0);
      }
      cp_async_commit();
      // while the rows are on their way: the row ids of the set's next tile
      uint32_t rid_n = 0u, vm_n = 0u;
      if (j + SETS < ntiles) lookup(j + SETS, rid_n, vm_n);
      // the rows have landed: made visible to the tensor core, then signalled
      cp_async_wait<0>();
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_full + 8 * stage);
      rid = rid_n;
      vm = vm_n;
    }
    if (aborted && lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
  } else if (warp == Shape::kQKWarp) {
    // ---------------- S = K Q^T: one thread, one tile ahead of the softmax groups
    if (lane == 0) {
      const uint64_t qd = umma_desc(q_smem);
      for (int j = 0; j < ntiles; ++j) {
        const int a = j & 1;
        bool ok = true;
        if (j >= 2) ok = mbar_wait(bar_sempty + 8 * a, ((j >> 1) - 1) & 1, &sh_abort);
        if (ok) ok = mbar_wait(bar_full + 8 * (j % kGUVStages), (j / kGUVStages) & 1, &sh_abort);
        if (!ok) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; break; }
        tc_fence_after();
        const uint64_t kd = umma_desc(smem0 + (uint32_t)(j % kGUKStages) * kGUTileBytes);
        const uint32_t d = tmem0 + (uint32_t)(a * kSUHeads);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          const uint64_t ka = kd + (uint64_t)((ks >> 2) * (kGUHalfBytes >> 4) + (ks & 3) * 2);
          const uint64_t qb = qd + (uint64_t)((ks >> 2) * ((kSUHeads * 128) >> 4) + (ks & 3) * 2);
          umma_bf16(d, ka, qb, kGUIdescQK, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar_kempty + 8 * (j % kGUKStages));   // the K stage may be refilled
        umma_commit(bar_sfull + 8 * a);
      }
    }
  } else {
    // ---------------- O_a^T += V^T P^T: one thread
    if (lane == 0 && ntiles > 0) {
      bool ok = true;
      for (int j = 0; j < ntiles; ++j) {
        const int stage = j % kGUVStages, a = j & 1;
        ok = mbar_wait(bar_pfull + 8 * a, (j >> 1) & 1, &sh_abort);
        if (!ok) break;
        tc_fence_after();
        const uint64_t vd = umma_desc_mn(v_ring + (uint32_t)stage * kGUTileBytes);
        const uint64_t pd = umma_desc(p_smem + a * kGUQBytes);
        const uint32_t d = tmem0 + (uint32_t)((2 + (G == 2 ? a : 0)) * kSUHeads);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          // 16 keys further: sixteen 128-byte rows of the V tile, 32 bytes along a row of the P tile
          const uint64_t va = vd + (uint64_t)(ks * ((16 * 128) >> 4));
          const uint64_t pb = pd + (uint64_t)((ks >> 2) * ((kSUHeads * 128) >> 4) + (ks & 3) * 2);
          umma_bf16(d, va, pb, kGUIdescPV, (j >= G || ks > 0) ? 1u : 0u);
        }
        umma_commit(bar_vempty + 8 * stage);   // the V stage may be refilled
        umma_commit(bar_pempty + 8 * a);       // and the group's P tile
      }
      if (ok) umma_commit(bar_odone);
      else { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (sh_abort) {
    // MMAs may still be in flight: a bounded wait on a last commit of each issuing thread before the
    // tensor memory goes back
    if (tid == Shape::kQKWarp * 32 || tid == Shape::kPVWarp * 32) {
      const uint32_t bar = bar_drain + 8 * (warp - Shape::kQKWarp);
      umma_commit(bar);
      const long long t0 = clock64();
      while (!mbar_try_wait(bar, 0))
        if (clock64() - t0 > kWaitBudgetCycles / 8) break;
    }
    __syncthreads();
  }
  if (warp == Shape::kQKWarp) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem0), "r"((uint32_t)kGUTmemCols) : "memory");
  }
}

}  // namespace prhs
