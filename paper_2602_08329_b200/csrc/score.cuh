// Retrieval pass, part 1: dense logits a_i = q . k_i / sqrt(d) for every cached position
// (Eq. 2), written as fp32 scores, plus per-chunk online log-sum-exp partials.
//
// The K stream goes straight from global memory into tensor-core operand registers: with
// keys as the N dimension of mma.sync m16n8k16 and the (up to 16) query heads of one KV
// head as the M dimension, lane (g, tg) needs elements of key row g only, and because a dot
// product does not care in which order the 128 dimensions are visited, the lane may take
// whole 16-byte chunks (chunk tg + 4j, j = 0..3) and call their elements k-slots of its own
// choosing, as long as the query fragments use the same assignment.  No shared-memory
// staging, no ldmatrix: 4 coalesced 16-byte loads and 8 MMAs per 8 keys, for every group
// size from MHA (1 head) to 16 heads.
#pragma once
#include "common.cuh"

namespace prhs {

constexpr int kScoreThreads = 256;
constexpr int kScoreWarps = kScoreThreads / 32;
constexpr int kScoreTilesPerIter = 4;           // 4 n-tiles = 32 keys = 8 KB in flight per warp

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Persistent CTAs: grid.x CTAs share the work items (unit, chunk) -- unit = (b, kvh), chunk =
// chunk_rows consecutive keys -- in unit-major order, each CTA taking one contiguous range, so
// that the grid is exactly one wave and the query fragments are reloaded only when the unit
// changes.  Dynamic shared memory: (batch + 1) ints.  chunk_rows: a multiple of 256 (8 warps
// x 32 keys).
__global__ void __launch_bounds__(kScoreThreads, 2)
score_mma_kernel(const __nv_bfloat16* __restrict__ q, KvDev kv, float* __restrict__ scores, int ld,
                 float2* __restrict__ part_ml, int nchunks, int chunk_rows, int num_q_heads,
                 int num_kv_heads, int batch, int write_scores, uint32_t* flags) {
  extern __shared__ __align__(16) uint32_t sh_dyn[];
  const int group_size = num_q_heads / num_kv_heads;
  int* cum = reinterpret_cast<int*>(sh_dyn);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, tg = lane & 3;
  const bool has0 = g < group_size, has1 = g + 8 < group_size;

  // items per sequence: Hkv * ceil(t_b / chunk_rows); exclusive prefix in cum[0..batch]
  for (int b = tid; b < batch; b += kScoreThreads) {
    const int t = __ldg(kv.seq_lens + b);
    cum[b + 1] = num_kv_heads * ((max(t, 0) + chunk_rows - 1) / chunk_rows);
  }
  __syncthreads();
  if (tid == 0) {
    cum[0] = 0;
    for (int b = 0; b < batch; ++b) cum[b + 1] += cum[b];
  }
  __syncthreads();
  const int total_items = cum[batch];
  const int item0 = (int)(((long long)total_items * blockIdx.x) / gridDim.x);
  const int item1 = (int)(((long long)total_items * (blockIdx.x + 1)) / gridDim.x);

  __shared__ float sm_m[kScoreWarps][16], sm_l[kScoreWarps][16];
  int b = 0;
  int cur_unit = -1;       // unit whose query fragments are loaded
  uint32_t a[8][4];

  for (int item = item0; item < item1; ++item) {
    while (cum[b + 1] <= item) ++b;
    const int t = __ldg(kv.seq_lens + b);
    const int nch_b = (t + chunk_rows - 1) / chunk_rows;
    const int local = item - cum[b];
    const int kvh = local / nch_b;
    const int chunk = local - kvh * nch_b;
    const int unit = b * num_kv_heads + kvh;
    const int head0 = kvh * group_size;
    const int row0 = chunk * chunk_rows;
    const int row1 = min(row0 + chunk_rows, t);
    const int span = chunk_rows / kScoreWarps;
    const int wrow0 = row0 + warp * span;
    const int wrow1 = min(wrow0 + span, row1);

    if (unit != cur_unit) {
      cur_unit = unit;
  // query fragments: k-step 2j uses elements 8c..8c+3 of chunk c = tg + 4j, k-step 2j+1 the rest
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    uint4 x0 = make_uint4(0u, 0u, 0u, 0u), x1 = x0;
    const long long qo = ((long long)b * num_q_heads + head0) * kHeadDim + (tg + 4 * j) * 8;
    if (has0) x0 = *reinterpret_cast<const uint4*>(q + qo + (long long)g * kHeadDim);
    if (has1) x1 = *reinterpret_cast<const uint4*>(q + qo + (long long)(g + 8) * kHeadDim);
    a[2 * j][0] = x0.x; a[2 * j][1] = x1.x; a[2 * j][2] = x0.y; a[2 * j][3] = x1.y;
    a[2 * j + 1][0] = x0.z; a[2 * j + 1][1] = x1.z; a[2 * j + 1][2] = x0.w; a[2 * j + 1][3] = x1.w;
  }
    }   // unit change

  // paged cache: the 16 pages of this warp's span, one per lane
  int pg = 0;
  if (kv.page_table != nullptr && lane < 16 && wrow0 + lane * 16 < wrow1) {
    pg = __ldg(kv.page_table + (long long)b * kv.page_table_stride + (wrow0 >> kPageShift) + lane);
    if ((unsigned)pg >= (unsigned)kv.num_pages) {
      atomicOr(flags, kFlagBadPage);
      pg = -1;
    }
  }
  const long long head_off = (long long)kvh * kv.stride_head + tg * 8;
  const long long seq_off = (long long)b * kv.stride_outer;

  float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;   // heads g and g + 8

  for (int it = wrow0; it < wrow1; it += 8 * kScoreTilesPerIter) {
    uint4 kx[kScoreTilesPerIter][4];
#pragma unroll
    for (int tile = 0; tile < kScoreTilesPerIter; ++tile) {
      const int row = it + tile * 8 + g;
      long long off = -1;
      if (kv.page_table != nullptr) {
        const int page = __shfl_sync(0xffffffffu, pg, ((it + tile * 8) - wrow0) >> kPageShift);
        if (row < wrow1 && page >= 0)
          off = (long long)page * kv.stride_outer + head_off + (long long)(row & 15) * kHeadDim;
      } else if (row < wrow1) {
        off = seq_off + head_off + (long long)row * kHeadDim;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        kx[tile][j] = off >= 0 ? ldg_stream(kv.k + off + 32 * j) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int tile = 0; tile < kScoreTilesPerIter; ++tile) {
      float c[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        mma_bf16_16816(c, a[2 * j], kx[tile][j].x, kx[tile][j].y);
        mma_bf16_16816(c, a[2 * j + 1], kx[tile][j].z, kx[tile][j].w);
      }
      // lane (g, tg) holds keys key0, key0 + 1 for heads g (c[0], c[1]) and g + 8 (c[2], c[3])
      const int key0 = it + tile * 8 + 2 * tg;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        if (hh == 0 ? has0 : has1) {
          const int head = head0 + g + 8 * hh;
          const float s0 = c[2 * hh] * kScale, s1 = c[2 * hh + 1] * kScale;
          float& m = hh == 0 ? m0 : m1;
          float& l = hh == 0 ? l0 : l1;
          float* dst = scores + ((long long)b * num_q_heads + head) * ld + key0;
          if (key0 + 1 < wrow1) {
            if (write_scores) *reinterpret_cast<float2*>(dst) = make_float2(s0, s1);
            const float x0 = s0 * kLog2e, x1 = s1 * kLog2e;
            const float mn = fmaxf(m, fmaxf(x0, x1));
            l = l * exp2f(m - mn) + exp2f(x0 - mn) + exp2f(x1 - mn);
            m = mn;
          } else if (key0 < wrow1) {
            if (write_scores) dst[0] = s0;
            const float x0 = s0 * kLog2e;
            const float mn = fmaxf(m, x0);
            l = l * exp2f(m - mn) + exp2f(x0 - mn);
            m = mn;
          }
        }
      }
    }
  }

  // ---- reduce (m, l) per head: over the 4 lanes of a group, then over the warps
#pragma unroll
  for (int off = 1; off <= 2; off <<= 1) {
    float m2 = __shfl_xor_sync(0xffffffffu, m0, off), l2 = __shfl_xor_sync(0xffffffffu, l0, off);
    ml_combine(m0, l0, m2, l2);
    m2 = __shfl_xor_sync(0xffffffffu, m1, off);
    l2 = __shfl_xor_sync(0xffffffffu, l1, off);
    ml_combine(m1, l1, m2, l2);
  }
  __syncthreads();           // the previous item's partials have been read
  if (tg == 0) {
    sm_m[warp][g] = m0; sm_l[warp][g] = l0;
    sm_m[warp][g + 8] = m1; sm_l[warp][g + 8] = l1;
  }
  __syncthreads();
  if (tid < group_size) {
    float mm = -INFINITY, ll = 0.f;
    for (int w = 0; w < kScoreWarps; ++w) ml_combine(mm, ll, sm_m[w][tid], sm_l[w][tid]);
    part_ml[((long long)b * num_q_heads + head0 + tid) * nchunks + chunk] = make_float2(mm, ll);
  }
  }   // items

}

}  // namespace prhs
