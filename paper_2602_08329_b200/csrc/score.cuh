// Retrieval pass, part 1: dense logits a_i = q . k_i / sqrt(d) for every cached position
// (Eq. 2), written as fp32 scores, plus per-chunk online log-sum-exp partials.
#pragma once
#include "common.cuh"

namespace prhs {

constexpr int kScoreThreads = 256;       // 16 half-warps; one half-warp covers one 256 B row
constexpr int kScoreRowsPerIter = 256;   // 16 half-warps x 16 rows

// grid (nchunks, Hq / GQ, B).  Each CTA streams `chunk_rows` keys of one KV head once and
// scores them against GQ query heads of that head's group.  Half-warp lane j holds elements
// [8j, 8j+8) of the row; a block of 16 rows is buffered so that each head's scores leave as
// one 64-byte store.
template <int GQ>
__global__ void __launch_bounds__(kScoreThreads)
score_kernel(const __nv_bfloat16* __restrict__ q, KvDev kv, float* __restrict__ scores, int ld,
             float2* __restrict__ part_ml, int nchunks, int chunk_rows, int num_q_heads,
             int group_size, int write_scores, uint32_t* flags) {
  const int b = blockIdx.z;
  const int head0 = blockIdx.y * GQ;
  const int kvh = head0 / group_size;
  const int chunk = blockIdx.x;
  const int t = __ldg(kv.seq_lens + b);
  const int row0 = chunk * chunk_rows;
  const int row1 = min(row0 + chunk_rows, t);
  const int tid = threadIdx.x;
  const int l16 = tid & 15;
  const int hw = tid >> 4;

  float qf[GQ][8];
#pragma unroll
  for (int h = 0; h < GQ; ++h) {
    const uint4 x = *reinterpret_cast<const uint4*>(
        q + ((long long)b * num_q_heads + head0 + h) * kHeadDim + l16 * 8);
    qf[h][0] = bf_lo(x.x); qf[h][1] = bf_hi(x.x); qf[h][2] = bf_lo(x.y); qf[h][3] = bf_hi(x.y);
    qf[h][4] = bf_lo(x.z); qf[h][5] = bf_hi(x.z); qf[h][6] = bf_lo(x.w); qf[h][7] = bf_hi(x.w);
  }
  float m[GQ], l[GQ];
#pragma unroll
  for (int h = 0; h < GQ; ++h) { m[h] = -INFINITY; l[h] = 0.f; }

  // the trip count is uniform over a warp (its two half-warps take adjacent 16-row blocks)
  for (int wbase = row0 + (tid >> 5) * 32; wbase < row1; wbase += kScoreRowsPerIter) {
    const int blk = wbase + (hw & 1) * 16;
    float keep[GQ];
#pragma unroll
    for (int h = 0; h < GQ; ++h) keep[h] = 0.f;
#pragma unroll
    for (int e0 = 0; e0 < 16; e0 += 8) {
      uint4 kx[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int row = blk + e0 + u;
        kx[u] = make_uint4(0u, 0u, 0u, 0u);
        if (row < row1) {
          const long long off = row_offset(kv, b, kvh, row, flags);
          if (off >= 0) kx[u] = ldg_stream(kv.k + off + l16 * 8);
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
#pragma unroll
        for (int h = 0; h < GQ; ++h) {
          const float s = half_warp_sum(dot8(kx[u], qf[h])) * kScale;
          if (l16 == e0 + u) keep[h] = s;
        }
      }
    }
    const int row = blk + l16;
    if (row < row1) {
#pragma unroll
      for (int h = 0; h < GQ; ++h) {
        if (write_scores)
          scores[((long long)b * num_q_heads + head0 + h) * ld + row] = keep[h];
        const float x = keep[h] * kLog2e;
        const float mn = fmaxf(m[h], x);
        l[h] = l[h] * exp2f(m[h] - mn) + exp2f(x - mn);
        m[h] = mn;
      }
    }
  }

  // reduce (m, l) over the CTA, one pair per head
  __shared__ float sm_m[kScoreThreads / 32][GQ];
  __shared__ float sm_l[kScoreThreads / 32][GQ];
#pragma unroll
  for (int h = 0; h < GQ; ++h) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m[h], off);
      const float l2 = __shfl_xor_sync(0xffffffffu, l[h], off);
      ml_combine(m[h], l[h], m2, l2);
    }
    if ((tid & 31) == 0) { sm_m[tid >> 5][h] = m[h]; sm_l[tid >> 5][h] = l[h]; }
  }
  __syncthreads();
  if (tid < GQ) {
    float mm = -INFINITY, ll = 0.f;
    for (int w = 0; w < kScoreThreads / 32; ++w) ml_combine(mm, ll, sm_m[w][tid], sm_l[w][tid]);
    part_ml[((long long)b * num_q_heads + head0 + tid) * nchunks + chunk] = make_float2(mm, ll);
  }
}

}  // namespace prhs
