// Retrieval scoring with the K stream staged by TMA (contiguous and paged caches).
//
// Logits a_i = q . k_i / sqrt(d) for all i < t (Eq. 2), as in score_ring_kernel, but the K
// tiles are brought into shared memory by the tensor memory accelerator: one elected thread
// issues two `cp.async.bulk.tensor.2d` copies per 64-key stage (a [64 rows][64 columns] box for
// each half of the 128 dimensions, 128-byte swizzle so that ldmatrix reads are conflict-free),
// completion is signalled on an mbarrier, and eight consumer warps (8 keys each) run the
// m16n8k16 MMAs for all heads of the KV group.  A six-stage ring keeps up to 80 KB in flight
// per CTA with no address arithmetic in the consumer warps.  With a paged cache the tensor is
// the page pool, a stage is four pages of 16 keys, and eight lanes of the producer warp each
// look a page id up and issue one [16 rows][64 columns] box (ids of the next stage are fetched
// while the current one is issued); pages past the end of the sequence are not fetched and an
// id outside the pool is skipped and flagged.
//
// Every wait on an mbarrier is bounded: a wait that exceeds its budget records
// kFlagTimeout and the CTA drains and returns, so a wrong descriptor cannot hang the GPU.
#pragma once
#include <cuda.h>

#include "attn.cuh"
#include "common.cuh"

namespace prhs {

constexpr int kSTConsumers = 8;                         // consumer warps
constexpr int kSTNT = 64 / (8 * kSTConsumers);          // 8-key MMA n-tiles per warp and stage
constexpr int kSTThreads = (kSTConsumers + 1) * 32;     // + one producer warp
constexpr int kSTStageRows = 64;                        // keys per stage
constexpr int kSTHalfBytes = kSTStageRows * 128;        // one [64][64] bf16 box = 8 KB
constexpr int kSTStageBytes = 2 * kSTHalfBytes;         // 16 KB
constexpr int kSTStages = 6;
constexpr int kSTSmemBytes = kSTStages * kSTStageBytes + 1024;   // + slack to align to 1 KB
constexpr uint32_t kFlagTimeout = 8u;
constexpr long long kWaitBudgetCycles = 4000000000ll;   // about two seconds

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait: false if the phase did not complete within the cycle budget, or if another
// thread of the CTA has already given up (*abort != 0).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const volatile int* abort,
                                          long long budget = kWaitBudgetCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (*abort || clock64() - t0 > budget) return false;
  return true;
}
// The key stream is read once and is far larger than L2: its lines are marked evict-first, and
// the logits (a few tens of MB that the selection kernel reads next) evict-last, so that the
// stream does not push the logits out to DRAM before they are used.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void st_f32x2_hint(float* p, float a, float b, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1, %2}, %3;" ::"l"(p), "f"(a), "f"(b), "l"(policy) : "memory");
}
__device__ __forceinline__ void st_f32_hint(float* p, float a, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.f32 [%0], %1, %2;" ::"l"(p), "f"(a), "l"(policy) : "memory");
}

// grid (splits, Hkv, B).  tm_k: K viewed as [rows][128] bf16 (row pitch 256 B), 128-byte swizzle.
// Contiguous: box [64][64], row of (b, kvh, i) = b * outer_rows + kvh * head_rows + i.
// Paged: box [16][64], row of (page, kvh, i mod 16) = page * outer_rows + kvh * head_rows + i mod 16.
template <bool kPaged>
__global__ void __launch_bounds__(kSTThreads)
score_tma_kernel(const __grid_constant__ CUtensorMap tm_k, ScoreParams p) {
  extern __shared__ unsigned char st_smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kSTStages];     // full[0..NS), empty[NS..2NS)
  __shared__ float sm_m[kSTConsumers][16], sm_l[kSTConsumers][16];
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
  const int g = lane >> 2, tg = lane & 3;
  const int t = __ldg(p.kv.seq_lens + b);
  // Equal-sized chunks of rows (a multiple of the stage) for every sequence: a short sequence of
  // a ragged batch fills fewer CTAs instead of many short ones; the others leave at once.
  int per = p.chunk_rows;
  if (per <= 0) {
    per = (t + p.splits - 1) / p.splits;
    per = (per + kSTStageRows - 1) & ~(kSTStageRows - 1);
  }
  if (split * per >= t && split > 0) {
    if ((int)threadIdx.x < gq)
      p.part_ml[((long long)b * p.num_q_heads + head0 + threadIdx.x) * p.splits + split] = make_float2(-INFINITY, 0.f);
    return;
  }
  const int start = min(split * per, t);
  const int end = min(start + per, t);
  const int nstages = (end - start + kSTStageRows - 1) / kSTStageRows;
  const uint32_t smem0 = ((uint32_t)__cvta_generic_to_shared(st_smem_raw) + 1023u) & ~1023u;
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars);
  const int outer_rows = (int)(p.kv.stride_outer >> 7), head_rows = (int)(p.kv.stride_head >> 7);
  const int row_base = kPaged ? kvh * head_rows : b * outer_rows + kvh * head_rows + start;

  if (tid == 0) {
    for (int s = 0; s < kSTStages; ++s) {
      mbar_init(bar0 + 8 * s, 1);                          // full: the producer's expect_tx arrive
      mbar_init(bar0 + 8 * (kSTStages + s), kSTConsumers); // empty: one arrive per consumer warp
    }
    sh_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();

  if (warp == kSTConsumers) {
    // ---------------- producer: one elected lane feeds the ring (contiguous cache); with a paged
    // cache lanes 0-7 each look up one of the stage's four pages and fetch one half of it
    const uint64_t pol_k = l2_policy_evict_first();
    if (!kPaged) {
      if (lane == 0) {
        for (int j = 0; j < nstages; ++j) {
          const int slot = j % kSTStages;
          if (j >= kSTStages && !mbar_wait(bar0 + 8 * (kSTStages + slot), ((j / kSTStages) - 1) & 1, &sh_abort)) {
            atomicOr(p.flags, kFlagTimeout);
            sh_abort = 1;
            break;
          }
          if (*(volatile int*)&sh_abort) break;
          const uint32_t full = bar0 + 8 * slot;
          const uint32_t dst = smem0 + slot * kSTStageBytes;
          mbar_expect_tx(full, kSTStageBytes);
          tma_load_2d(dst, &tm_k, 0, row_base + j * kSTStageRows, full, pol_k);
          tma_load_2d(dst + kSTHalfBytes, &tm_k, 64, row_base + j * kSTStageRows, full, pol_k);
        }
      }
    } else {
      const int x = (lane >> 1) & 3, half = lane & 1;   // lanes 0-7: page x of the stage, 64-column half
      const int* ptab = p.kv.page_table + (long long)b * p.kv.page_table_stride + (start >> kPageShift) + x;
      bool have_next = lane < 8 && start + 16 * x < end;
      int pg_next = have_next ? __ldg(ptab) : 0;
      for (int j = 0; j < nstages; ++j) {
        const int slot = j % kSTStages;
        const int pg = pg_next;
        const bool have = have_next;                // false: past the end, or lane >= 8
        // page id of the next stage, in flight during the wait below
        have_next = lane < 8 && j + 1 < nstages && start + (j + 1) * kSTStageRows + 16 * x < end;
        pg_next = have_next ? __ldg(ptab + 4 * (j + 1)) : 0;
        bool ok = true;
        if (lane == 0 && j >= kSTStages)
          ok = mbar_wait(bar0 + 8 * (kSTStages + slot), ((j / kSTStages) - 1) & 1, &sh_abort);
        if (lane == 0 && !ok) {
          atomicOr(p.flags, kFlagTimeout);
          sh_abort = 1;
        }
        __syncwarp();
        if (*(volatile int*)&sh_abort) break;       // warp-uniform: read after the barrier above
        const bool fetch = have && (unsigned)pg < (unsigned)p.kv.num_pages;
        if (have && !fetch) atomicOr(p.flags, kFlagBadPage);
        const uint32_t okmask = __ballot_sync(0xffffffffu, fetch);
        const uint32_t full = bar0 + 8 * slot;
        // the barrier needs its arrive even when no page of the stage is fetched
        if (lane == 0) mbar_expect_tx(full, (uint32_t)__popc(okmask) * 2048u);
        __syncwarp();
        if (fetch) {
          const uint32_t dst = smem0 + slot * kSTStageBytes + half * kSTHalfBytes + x * 2048;
          tma_load_2d(dst, &tm_k, 64 * half, pg * outer_rows + row_base, full, pol_k);
        }
      }
    }
  } else {
    // ---------------- consumers: 8 kSTNT keys of every stage per warp
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
    const uint64_t pol_s = l2_policy_evict_last();
    const int lm_mi = lane >> 3, lm_r = lane & 7;
    for (int j = 0; j < nstages; ++j) {
      const int slot = j % kSTStages;
      // every lane polls; the outcome is made uniform so that the warp leaves the loop together
      if (!__all_sync(0xffffffffu, mbar_wait(bar0 + 8 * slot, (j / kSTStages) & 1, &sh_abort))) {
        if (lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
        break;
      }
      const uint32_t kt = smem0 + slot * kSTStageBytes;
      const int pos0 = start + j * kSTStageRows + warp * (8 * kSTNT);
      float s[kSTNT][4];
#pragma unroll
      for (int nt = 0; nt < kSTNT; ++nt) { s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f; }
#pragma unroll
      for (int pp = 0; pp < 4; ++pp) {
        // logical 16-byte chunk 4pp + lm_mi of the 256-byte row: half = chunk / 8, c = chunk % 8
        const int chunk = 4 * pp + lm_mi;
        const uint32_t hb = kt + (chunk >> 3) * kSTHalfBytes + (((chunk & 7) ^ lm_r) << 4);
        uint32_t bk[kSTNT][4];
#pragma unroll
        for (int nt = 0; nt < kSTNT; ++nt) ldmatrix_x4(bk[nt], hb + (warp * (8 * kSTNT) + 8 * nt + lm_r) * 128);
#pragma unroll
        for (int nt = 0; nt < kSTNT; ++nt)
          mma_bf16_full(s[nt], aq[2 * pp][0], aq[2 * pp][1], aq[2 * pp][2], aq[2 * pp][3], bk[nt][0], bk[nt][1]);
#pragma unroll
        for (int nt = 0; nt < kSTNT; ++nt)
          mma_bf16_full(s[nt], aq[2 * pp + 1][0], aq[2 * pp + 1][1], aq[2 * pp + 1][2], aq[2 * pp + 1][3], bk[nt][2], bk[nt][3]);
      }
      // the tile has been read into registers: hand the slot back to the producer
      __syncwarp();
      if (lane == 0) mbar_arrive(bar0 + 8 * (kSTStages + slot));
      if (p.scores && p.group_max)
        store_group_max<kSTNT>(s, has0, has1, p.scores + ((long long)b * p.num_q_heads + head0) * p.ld, pos0, end);
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        if (hh == 0 ? has0 : has1) {
          float& m = hh == 0 ? m0 : m1;
          float& l = hh == 0 ? l0 : l1;
          float* dst = (p.scores && !p.group_max) ? p.scores + ((long long)b * p.num_q_heads + head0 + g + 8 * hh) * p.ld : nullptr;
#pragma unroll
          for (int nt = 0; nt < kSTNT; ++nt) {
            const int key0 = pos0 + 8 * nt + 2 * tg;
            const float s0 = s[nt][2 * hh] * kScale, s1 = s[nt][2 * hh + 1] * kScale;
            if (key0 + 1 < end) {
              if (dst) st_f32x2_hint(dst + key0, s0, s1, pol_s);
              const float x0 = s0 * kLog2e, x1 = s1 * kLog2e;
              const float mn = fmaxf(m, fmaxf(x0, x1));
              l = l * exp2f(m - mn) + exp2f(x0 - mn) + exp2f(x1 - mn);
              m = mn;
            } else if (key0 < end) {
              if (dst) st_f32_hint(dst + key0, s0, pol_s);
              const float x0 = s0 * kLog2e;
              const float mn = fmaxf(m, x0);
              l = l * exp2f(m - mn) + exp2f(x0 - mn);
              m = mn;
            }
          }
        }
      }
    }
#pragma unroll
    for (int off = 1; off <= 2; off <<= 1) {
      float m2 = __shfl_xor_sync(0xffffffffu, m0, off), l2 = __shfl_xor_sync(0xffffffffu, l0, off);
      ml_combine(m0, l0, m2, l2);
      m2 = __shfl_xor_sync(0xffffffffu, m1, off);
      l2 = __shfl_xor_sync(0xffffffffu, l1, off);
      ml_combine(m1, l1, m2, l2);
    }
    if (tg == 0) {
      sm_m[warp][g] = m0; sm_l[warp][g] = l0;
      sm_m[warp][g + 8] = m1; sm_l[warp][g + 8] = l1;
    }
  }
  __syncthreads();
  if (tid < gq) {
    float mm = -INFINITY, ll = 0.f;
    for (int w = 0; w < kSTConsumers; ++w) ml_combine(mm, ll, sm_m[w][tid], sm_l[w][tid]);
    p.part_ml[((long long)b * p.num_q_heads + head0 + tid) * p.splits + split] = make_float2(mm, ll);
  }
  // After an aborted wait some copies may still be in flight towards this CTA's shared
  // memory: give each full barrier one more bounded wait before the CTA returns.
  if (sh_abort && tid == 0) {
    for (int s = 0; s < kSTStages; ++s) {
      const long long t0 = clock64();
      while (!mbar_try_wait(bar0 + 8 * s, 0) && !mbar_try_wait(bar0 + 8 * s, 1))
        if (clock64() - t0 > kWaitBudgetCycles / 8) break;
    }
  }
}

// Self-test of the bounded wait: one thread waits on a barrier phase that nothing completes,
// with a short budget; the wait must come back false, and the kernel records kFlagTimeout the
// way the scoring kernel does.  Harmless by construction: the loop ends with the budget.
__global__ void wait_selftest_kernel(long long budget, uint32_t* flags, int* gave_up) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    const uint32_t b = (uint32_t)__cvta_generic_to_shared(&bar);
    mbar_init(b, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const bool ok = mbar_wait(b, 0, &abort_flag, budget);
    if (!ok) atomicOr(flags, kFlagTimeout);
    *gave_up = ok ? 0 : 1;
  }
}

}  // namespace prhs
