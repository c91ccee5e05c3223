// Measurement support: the bare row gather of the gathered attention, without its arithmetic.
//
// gather_probe_kernel fetches exactly the rows a prhs_sparse_decode_attn call would fetch (the K
// row and the V row of every list entry, 256 bytes each, addressed through the same view) with
// the work laid out like the attention kernel (one CTA of four warps per (sequence, head) unit
// and split, a warp per slice of the list, 16-entry stages), and does nothing with them beyond
// one shared-memory (or register) read per stage.  The fetch itself comes in four variants, so
// that the ceiling of each mechanism can be read next to the attention kernel's own time:
//   0  plain 16-byte read-only loads into registers, 8 rows in flight per half-warp
//   1  16-byte cp.async copies into a warp-private ring (what the attention kernel uses)
//   2  one 256-byte bulk copy (cp.async.bulk) per row, completion on an mbarrier
//   3  TMA row gather (cp.async.bulk.tensor.2d.tile::gather4): four rows per instruction
// No multicast anywhere; every mbarrier wait is bounded like the scoring kernel's.
#pragma once
#include <cuda.h>

#include "attn.cuh"
#include "common.cuh"
#include "score_tma.cuh"

namespace prhs {

constexpr int kGPStages = 3;
constexpr int kGPStageRows = 16;
constexpr int kGPStageBytes = 2 * kGPStageRows * kRowBytes;          // K rows + V rows: 8 KB
constexpr int kGPSmemBytes = kTWarps * kGPStages * kGPStageBytes + 1024;

struct GatherProbeParams {
  KvDev kv;                 // contiguous view
  const int* idx;           // [B][Hq][idx_stride]
  const int* count;         // [B][Hq]
  int idx_stride, num_q_heads, group_size, splits;
  uint32_t* flags;
  unsigned int* sink;       // one word; written only if a checksum takes an impossible value
};

__device__ __forceinline__ void bulk_copy_row(uint32_t dst, const void* src, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 256, [%2];"
               ::"r"(dst), "l"(src), "r"(bar) : "memory");
}
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* tm, int col, int r0, int r1, int r2, int r3,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes"
      " [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
      ::"r"(dst), "l"(tm), "r"(col), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
      : "memory");
}

// grid (splits, Hq, B), 128 threads.  tm_k / tm_v: K and V viewed as [rows][128] bf16 with a box of
// one row (used by variant 3 only).
template <int kVariant>
__global__ void __launch_bounds__(kTThreads)
gather_probe_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                    GatherProbeParams p) {
  extern __shared__ unsigned char gp_smem_raw[];
  __shared__ __align__(8) unsigned long long bars[kTWarps * kGPStages];
  __shared__ int sh_abort;
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int unit = b * p.num_q_heads + h;
  const int kvh = h / p.group_size;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = __ldg(p.kv.seq_lens + b);
  const int cnt = min(__ldg(p.count + unit), p.idx_stride);
  int per = (cnt + p.splits * kTWarps - 1) / (p.splits * kTWarps);
  per = (per + kGPStageRows - 1) & ~(kGPStageRows - 1);
  const int start = min((split * kTWarps + warp) * per, cnt);
  const int end = min(start + per, cnt);
  const int nstages = (end - start + kGPStageRows - 1) / kGPStageRows;
  const int* list = p.idx + (long long)unit * p.idx_stride;
  const uint32_t base_row = (uint32_t)b * (uint32_t)(p.kv.stride_outer >> 7) + (uint32_t)kvh * (uint32_t)(p.kv.stride_head >> 7);
  const uint32_t smem0 = ((uint32_t)__cvta_generic_to_shared(gp_smem_raw) + 1023u) & ~1023u;
  const uint32_t ring = smem0 + warp * (kGPStages * kGPStageBytes);
  const uint32_t bar0 = (uint32_t)__cvta_generic_to_shared(bars) + 8 * warp * kGPStages;
  unsigned int acc = 0u;

  // row id of list entry j of this warp's slice (an entry outside [0, t) is replaced by row 0 and flagged)
  auto row_of = [&](int j) -> uint32_t {
    if (j >= end) return base_row;
    const int pos = __ldg(list + j);
    if ((unsigned)pos >= (unsigned)t) {
      atomicOr(p.flags, kFlagBadIndex);
      return base_row;
    }
    return base_row + (uint32_t)pos;
  };

  if (kVariant == 0) {
    // each half-warp reads whole rows: lanes 0-15 the K row, 16-31 the V row, 8 entries in flight
    const uint4* src = reinterpret_cast<const uint4*>(lane < 16 ? p.kv.k : p.kv.v) + (lane & 15);
    for (int j = start; j < end; j += 8) {
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t rid = row_of(min(j + u, end - 1));
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                     : "=r"(v[u].x), "=r"(v[u].y), "=r"(v[u].z), "=r"(v[u].w) : "l"(src + (size_t)rid * 16));
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) acc ^= v[u].x ^ v[u].w;
    }
  } else if (kVariant == 1) {
    const __nv_bfloat16* src_base = (lane < 16 ? p.kv.k : p.kv.v) + (lane & 15) * 8;
    const uint32_t dst_tile = lane < 16 ? 0u : (uint32_t)(kGPStageRows * kRowBytes);
    auto issue = [&](int s) {
      if (s < nstages) {
        const uint32_t mine = row_of(start + s * kGPStageRows + (lane & 15));
        const uint32_t slot = ring + (uint32_t)(s % kGPStages) * kGPStageBytes + dst_tile;
#pragma unroll
        for (int r = 0; r < kGPStageRows; ++r) {
          const uint32_t rid = __shfl_sync(0xffffffffu, mine, r);
          cp_async_16_full(slot + r * kRowBytes + ((uint32_t)(lane & 15) << 4), src_base + (size_t)rid * kHeadDim);
        }
      }
      cp_async_commit();
    };
#pragma unroll
    for (int s = 0; s < kGPStages - 1; ++s) issue(s);
    for (int i = 0; i < nstages; ++i) {
      cp_async_wait<kGPStages - 2>();
      __syncwarp();
      issue(i + kGPStages - 1);
      unsigned int x;
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x) : "r"(ring + (uint32_t)(i % kGPStages) * kGPStageBytes + lane * 4));
      acc ^= x;
    }
    cp_async_wait<0>();
  } else {
    // variants 2 and 3: copies issued by lanes of the warp itself, completion on one mbarrier per stage
    if (tid == 0) sh_abort = 0;
    if (lane == 0) {
      for (int s = 0; s < kGPStages; ++s) mbar_init(bar0 + 8 * s, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    auto issue = [&](int s) {
      if (s >= nstages) return;
      const uint32_t slot = ring + (uint32_t)(s % kGPStages) * kGPStageBytes;
      const uint32_t bar = bar0 + 8 * (s % kGPStages);
      const uint32_t mine = row_of(start + s * kGPStageRows + (lane & 15));
      if (lane == 0) mbar_expect_tx(bar, kGPStageBytes);
      __syncwarp();
      if (kVariant == 2) {
        // lane r copies the K row of entry r, lane 16 + r its V row
        const __nv_bfloat16* src = (lane < 16 ? p.kv.k : p.kv.v) + (size_t)mine * kHeadDim;
        bulk_copy_row(slot + (lane < 16 ? 0u : (uint32_t)(kGPStageRows * kRowBytes)) + (lane & 15) * kRowBytes, src, bar);
      } else {
        // lanes 0-3 gather four K rows each, lanes 16-19 four V rows each
        const int q4 = lane & 15;
        const uint32_t r0 = __shfl_sync(0xffffffffu, mine, (4 * q4) & 15), r1 = __shfl_sync(0xffffffffu, mine, (4 * q4 + 1) & 15);
        const uint32_t r2 = __shfl_sync(0xffffffffu, mine, (4 * q4 + 2) & 15), r3 = __shfl_sync(0xffffffffu, mine, (4 * q4 + 3) & 15);
        if (q4 < 4)
          tma_gather4(slot + (lane < 16 ? 0u : (uint32_t)(kGPStageRows * kRowBytes)) + q4 * 4 * kRowBytes,
                      lane < 16 ? &tm_k : &tm_v, 0, (int)r0, (int)r1, (int)r2, (int)r3, bar);
      }
    };
    for (int s = 0; s < kGPStages - 1; ++s) issue(s);
    for (int i = 0; i < nstages; ++i) {
      const int slot_i = i % kGPStages;
      if (!__all_sync(0xffffffffu, mbar_wait(bar0 + 8 * slot_i, (i / kGPStages) & 1, &sh_abort))) {
        if (lane == 0) { atomicOr(p.flags, kFlagTimeout); sh_abort = 1; }
        break;
      }
      unsigned int x;
      asm volatile("ld.shared.u32 %0, [%1];" : "=r"(x) : "r"(ring + (uint32_t)slot_i * kGPStageBytes + lane * 4));
      acc ^= x;
      __syncwarp();
      issue(i + kGPStages - 1);
    }
    // after an aborted wait copies may still be in flight towards this CTA's shared memory
    __syncthreads();
    if (sh_abort && lane == 0) {
      for (int s = 0; s < kGPStages; ++s) {
        const long long t0 = clock64();
        while (!mbar_try_wait(bar0 + 8 * s, 0) && !mbar_try_wait(bar0 + 8 * s, 1))
          if (clock64() - t0 > kWaitBudgetCycles / 8) break;
      }
    }
  }
  if (acc == 0x9e3779b9u && cnt < 0) *p.sink = acc;      // never true: keeps the reads alive
}

}  // namespace prhs
