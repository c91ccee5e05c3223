// Retrieval scoring on the fifth-generation tensor cores (tcgen05), K stream staged by TMA.
//
// The same computation as score_tma_kernel -- logits a_i = q . k_i / sqrt(d) for all i < t (Eq. 2),
// the fp32 logits for the selection kernel and a per-split (max, sum) partial of the full softmax --
// with the contraction issued by ONE thread: a 128-key K tile lands in shared memory in the
// 128-byte-swizzled K-major layout the tensor core reads directly (two [128 rows][64 columns] TMA
// boxes, or sixteen [16][64] page boxes), the heads of the KV group sit in a 16-row Q tile of the
// same layout, and eight tcgen05.mma (M = 128 keys, N = 16 heads, K = 16) accumulate the tile's
// logits into tensor memory.  Four epilogue warps read their 32 lanes of the accumulator
// (tcgen05.ld, one key per thread, the group's heads across its registers), store the logits
// (consecutive lanes = consecutive keys: full 128-byte lines) and keep a running (max, sum) per
// head.  No ldmatrix, no per-warp MMA issue, no address arithmetic on the key rows: six warps per
// CTA instead of nine, and two accumulators in tensor memory let the MMAs of tile j + 1 run while
// tile j is read out.  The kernel is bound by the key stream exactly like score_tma_kernel (the two
// measure within 1 % of each other on every benchmark shape, this one ahead); it is the default
// because it leaves the SM's issue slots and registers nearly idle.  Not for cosine-gated steps, whose
// CTAs mostly return at once: CTAs of this kernel are several times slower to launch and retire than
// those of the mma.sync kernel even then (8448 empty CTAs: 28 us against 7 us).
//
// Warp roles: 0 = TMA producer, 1 = tensor-memory allocation + MMA issue, 2..5 = epilogue (tensor
// memory lanes 32 (warp mod 4) .. + 31).  Every mbarrier wait is bounded like score_tma_kernel's;
// the CTA frees its tensor memory on every path that allocated it.
#pragma once
#include <cuda.h>

#include "attn.cuh"
#include "common.cuh"
#include "score_tma.cuh"

namespace prhs {

constexpr int kSUTileRows = 128;                         // keys per MMA tile and ring stage
constexpr int kSUHalfBytes = kSUTileRows * 128;          // one [128][64] bf16 box = 16 KB
constexpr int kSUStageBytes = 2 * kSUHalfBytes;          // 32 KB
// Two stages of 32 KB: three CTAs fit on an SM, and a CTA that starts (tensor-memory allocation, Q tile,
// first copies) or ends is covered by the two others.  Deeper rings with fewer resident CTAs measured
// slower (three stages, two CTAs: +2 % with grouped queries; six stages, one CTA: +12 to +40 %).
constexpr int kSUStages = 2;
constexpr int kSUHeads = 16;                             // N of the MMA: heads of a KV group, zero-padded
constexpr int kSUQBytes = 2 * kSUHeads * 128;            // Q tile: two 64-column halves of 16 rows
constexpr int kSUThreads = 6 * 32;
constexpr int kSUSmemBytes = kSUStages * kSUStageBytes + kSUQBytes + 1024;
constexpr int kSUTmemCols = 32;                          // two accumulators of 16 fp32 columns
// instruction descriptor: D = fp32, A = B = bf16, both K-major, N = 16 (>> 3), M = 128 (>> 4)
constexpr uint32_t kSUIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kSUHeads >> 3) << 17) |
                              ((uint32_t)(kSUTileRows >> 4) << 24);
// shared-memory matrix descriptor, upper word: 8-row groups 1024 bytes apart, descriptor version 1,
// 128-byte swizzle; lower word: address >> 4 and a leading offset of one 16-byte unit
constexpr uint32_t kSUDescHi = 64u | (1u << 14) | (2u << 29);

__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  return ((uint64_t)kSUDescHi << 32) | (uint64_t)(((smem_addr >> 4) & 0x3fffu) | (1u << 16));
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the mbarrier receives one arrive when every MMA this thread issued before has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  // the registers are operands of the wait so that no use of them can be scheduled before it
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                 "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// grid (splits, Hkv, B), 192 threads.  tm_k: K viewed as [rows][128] bf16 (row pitch 256 B), 128-byte
// swizzle.  Contiguous: box [128][64]; paged: box [16][64] (one page).
template <bool kPaged>
__global__ void __launch_bounds__(kSUThreads)
score_umma_kernel(const __grid_constant__ CUtensorMap tm_k, ScoreParams p) {
  extern __shared__ unsigned char su_smem_raw[];
  // full[0..S), empty[S..2S), acc_full[2S..2S+2), acc_empty[2S+2..2S+4), drain[2S+4]
  __shared__ __align__(8) unsigned long long bars[2 * kSUStages + 5];
  __shared__ float sm_m[4][kSUHeads], sm_l[4][kSUHeads];
  __shared__ uint32_t tmem_slot;
  __shared__ int sh_abort;
  const int split = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int gq = p.group_size;
  const int head0 = kvh * gq;
  if (p.need != nullptr) {
    bool any = false;
    for (int j = 0; j < gq; ++j) any |= __ldg(p.need + b * p.num_q_heads + head0 + j) != 0;
    if (!any) return;
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = __ldg(p.kv.seq_lens + b);
  int per = p.chunk_rows;
  if (per <= 0) {
    per = (t + p.splits - 1) / p.splits;
    per = (per + kSUTileRows - 1) & ~(kSUTileRows - 1);
  }
  if (split * per >= t && split > 0) {
    if ((int)threadIdx.x < gq)
      p.part_ml[((long long)b * p.num_q_heads + head0 + threadIdx.x) * p.splits + split] = make_float2(-INFINITY, 0.f);
    return;
  }
  const int start = min(split * per, t);
  const int end = min(start + per, t);
  const int ntiles = (end - start + kSUTileRows - 1) / kSUTileRows;
  const uint32_t smem0 = ((uint32_t)__cvta_generic_to_shared(su_smem_raw) + 1023u) & ~1023u;
  const uint32_t q_smem = smem0 + kSUStages * kSUStageBytes;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  const uint32_t bar_full = bar0, bar_empty = bar0 + 8 * kSUStages;
  const uint32_t bar_afull = bar0 + 8 * (2 * kSUStages), bar_aempty = bar_afull + 16, bar_drain = bar_afull + 32;
  const int outer_rows = (int)(p.kv.stride_outer >> 7), head_rows = (int)(p.kv.stride_head >> 7);
  const int row_base = kPaged ? kvh * head_rows : b * outer_rows + kvh * head_rows + start;

  if (tid == 0) {
    for (int s = 0; s < kSUStages; ++s) {
      mbar_init(bar_full + 8 * s, 1);      // the producer's expect_tx arrive
      mbar_init(bar_empty + 8 * s, 1);     // one commit of the MMA thread
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(bar_afull + 8 * a, 1);     // one commit of the MMA thread
      mbar_init(bar_aempty + 8 * a, 4);    // one arrive per epilogue warp
    }
    mbar_init(bar_drain, 1);
    sh_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // Q tile: head row h, 16-byte chunk c of half hf at  hf * 2048 + h * 128 + ((c ^ (h & 7)) << 4)
  // (rows of heads the group does not have are zero)
  for (int i = tid; i < kSUHeads * 16; i += kSUThreads) {
    const int h = i >> 4, c16 = i & 15, hf = c16 >> 3, c = c16 & 7;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (h < gq)
      v = __ldg(reinterpret_cast<const uint4*>(p.q + ((long long)b * p.num_q_heads + head0 + h) * kHeadDim) + c16);
    const uint32_t dst = q_smem + hf * (kSUHeads * 128) + h * 128 + ((c ^ (h & 7)) << 4);
    asm volatile("st.shared.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                 ::"r"((uint32_t)__cvta_generic_to_shared(&tmem_slot)), "r"((uint32_t)kSUTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem0 = *(volatile uint32_t*)&tmem_slot;

  if (warp == 0) {
    // ---------------- producer
    const uint64_t pol_k = l2_policy_evict_first();
    if (!kPaged) {
      if (lane == 0) {
        for (int j = 0; j < ntiles; ++j) {
          const int slot = j % kSUStages;
          if (j >= kSUStages && !mbar_wait(bar_empty + 8 * slot, ((j / kSUStages) - 1) & 1, &sh_abort)) {
            atomicOr(p.flags, kFlagTimeout);
            sh_abort = 1;
            break;
          }
          if (*(volatile int*)&sh_abort) break;
          const uint32_t full = bar_full + 8 * slot;
          const uint32_t dst = smem0 + slot * kSUStageBytes;
          mbar_expect_tx(full, kSUStageBytes);
          tma_load_2d(dst, &tm_k, 0, row_base + j * kSUTileRows, full, pol_k);
          tma_load_2d(dst + kSUHalfBytes, &tm_k, 64, row_base + j * kSUTileRows, full, pol_k);
        }
      }
    } else {
      // lanes 0-15: page x of the tile's eight, 64-column half
      const int x = (lane >> 1) & 7, half = lane & 1;
      const int* ptab = p.kv.page_table + (long long)b * p.kv.page_table_stride + (start >> kPageShift) + x;
      bool have_next = lane < 16 && start + 16 * x < end;
      int pg_next = have_next ? __ldg(ptab) : 0;
      for (int j = 0; j < ntiles; ++j) {
        const int slot = j % kSUStages;
        const int pg = pg_next;
        const bool have = have_next;
        have_next = lane < 16 && j + 1 < ntiles && start + (j + 1) * kSUTileRows + 16 * x < end;
        pg_next = have_next ? __ldg(ptab + 8 * (j + 1)) : 0;
        bool ok = true;
        if (lane == 0 && j >= kSUStages) ok = mbar_wait(bar_empty + 8 * slot, ((j / kSUStages) - 1) & 1, &sh_abort);
        if (lane == 0 && !ok) {
          atomicOr(p.flags, kFlagTimeout);
          sh_abort = 1;
        }
        __syncwarp();
        if (*(volatile int*)&sh_abort) break;
        const bool fetch = have && (unsigned)pg < (unsigned)p.kv.num_pages;
        if (have && !fetch) atomicOr(p.flags, kFlagBadPage);
        const uint32_t okmask = __ballot_sync(0xffffffffu, fetch);
        const uint32_t full = bar_full + 8 * slot;
        if (lane == 0) mbar_expect_tx(full, (uint32_t)__popc(okmask) * 2048u);
        __syncwarp();
        if (fetch) {
          const uint32_t dst = smem0 + slot * kSUStageBytes + half * kSUHalfBytes + x * 2048;
          tma_load_2d(dst, &tm_k, 64 * half, pg * outer_rows + row_base, full, pol_k);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issue: one thread
    if (lane == 0) {
      const uint64_t qd = umma_desc(q_smem);
      for (int j = 0; j < ntiles; ++j) {
        const int slot = j % kSUStages, a = j & 1;
        bool ok = true;
        if (j >= 2) ok = mbar_wait(bar_aempty + 8 * a, ((j >> 1) - 1) & 1, &sh_abort);
        if (ok) ok = mbar_wait(bar_full + 8 * slot, (j / kSUStages) & 1, &sh_abort);
        if (!ok) {
          atomicOr(p.flags, kFlagTimeout);
          sh_abort = 1;
          break;
        }
        tc_fence_after();
        const uint64_t kd = umma_desc(smem0 + slot * kSUStageBytes);
        const uint32_t d = tmem0 + (uint32_t)(a * kSUHeads);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          // 16 columns = 32 bytes = two 16-byte units further along the swizzled row; the second
          // 64-column half is its own box
          const uint64_t ka = kd + (uint64_t)((ks >> 2) * (kSUHalfBytes >> 4) + (ks & 3) * 2);
          const uint64_t qb = qd + (uint64_t)((ks >> 2) * ((kSUHeads * 128) >> 4) + (ks & 3) * 2);
          umma_bf16(d, ka, qb, kSUIdesc, ks > 0 ? 1u : 0u);
        }
        umma_commit(bar_empty + 8 * slot);     // the stage may be refilled
        umma_commit(bar_afull + 8 * a);        // the accumulator may be read
      }
    }
  } else {
    // ---------------- epilogue: thread = one key of every tile
    const int sub = warp & 3;
    const int row = 32 * sub + lane;
    float m[kSUHeads], l[kSUHeads];
#pragma unroll
    for (int h = 0; h < kSUHeads; ++h) { m[h] = -INFINITY; l[h] = 0.f; }
    const uint64_t pol_s = l2_policy_evict_last();
    float* srow = p.scores ? p.scores + ((long long)b * p.num_q_heads + head0) * p.ld : nullptr;
    for (int j = 0; j < ntiles; ++j) {
      const int a = j & 1;
      if (!__all_sync(0xffffffffu, mbar_wait(bar_afull + 8 * a, (j >> 1) & 1, &sh_abort))) {
        if (lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
        break;
      }
      tc_fence_after();
      float s[16];
      tmem_ld16(tmem0 + ((uint32_t)(32 * sub) << 16) + (uint32_t)(a * kSUHeads), s);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_aempty + 8 * a);
      const int key = start + j * kSUTileRows + row;
      if (key < end) {
        if (srow && p.group_max) {
          float x = s[0];
#pragma unroll
          for (int h = 1; h < kSUHeads; ++h)
            if (h < gq) x = fmaxf(x, s[h]);
          st_f32_hint(srow + key, x * kScale, pol_s);
        }
#pragma unroll
        for (int h = 0; h < kSUHeads; ++h) {
          if (h < gq) {
            const float sc = s[h] * kScale;
            if (srow && !p.group_max) st_f32_hint(srow + (long long)h * p.ld + key, sc, pol_s);
            const float x = sc * kLog2e;
            const float mn = fmaxf(m[h], x);
            l[h] = l[h] * exp2f(m[h] - mn) + exp2f(x - mn);
            m[h] = mn;
          }
        }
      }
    }
#pragma unroll
    for (int h = 0; h < kSUHeads; ++h) {
      if (h < gq) {
        float mm = m[h], ll = l[h];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, mm, off), l2 = __shfl_xor_sync(0xffffffffu, ll, off);
          ml_combine(mm, ll, m2, l2);
        }
        if (lane == 0) { sm_m[sub][h] = mm; sm_l[sub][h] = ll; }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid < gq && !sh_abort) {
    float mm = -INFINITY, ll = 0.f;
    for (int w = 0; w < 4; ++w) ml_combine(mm, ll, sm_m[w][tid], sm_l[w][tid]);
    p.part_ml[((long long)b * p.num_q_heads + head0 + tid) * p.splits + split] = make_float2(mm, ll);
  }
  // After an aborted wait copies and MMAs may still be in flight: give each full barrier one more
  // bounded wait, and the tensor core a bounded wait on a last commit, before the tensor memory
  // is handed back.
  if (sh_abort) {
    if (tid == 0) {
      for (int s = 0; s < kSUStages; ++s) {
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_full + 8 * s, 0) && !mbar_try_wait(bar_full + 8 * s, 1))
          if (clock64() - t0 > kWaitBudgetCycles / 8) break;
      }
    }
    if (tid == 32) {
      umma_commit(bar_drain);
      const long long t0 = clock64();
      while (!mbar_try_wait(bar_drain, 0))
        if (clock64() - t0 > kWaitBudgetCycles / 8) break;
    }
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem0), "r"((uint32_t)kSUTmemCols) : "memory");
  }
}

}  // namespace prhs
