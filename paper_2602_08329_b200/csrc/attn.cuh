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
build_set_kernel(const int* __restrict__ mid, const int* __restrict__ n_mid, int mid_stride,
                 const int* __restrict__ seq_lens, int sinks, int window, int num_q_heads,
                 int* __restrict__ out_idx, int idx_stride, int* __restrict__ out_count) {
  const int unit = blockIdx.x;
  const int b = unit / num_q_heads;
  const int t = __ldg(seq_lens + b);
  const int* M = mid + (long long)unit * mid_stride;
  const int nm = __ldg(n_mid + unit);
  const int s0 = min(sinks, t);
  const int wlo = max(max(t - window, 0), s0);
  __shared__ int sh_lo, sh_hi;
  if (threadIdx.x < 2) {
    const int bound = threadIdx.x == 0 ? s0 : wlo;   // first entry >= bound
    int a = 0, c = nm;
    while (a < c) {
      const int mid_i = (a + c) >> 1;
      if (__ldg(M + mid_i) < bound) a = mid_i + 1; else c = mid_i;
    }
    if (threadIdx.x == 0) sh_lo = a; else sh_hi = a;
  }
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
constexpr int kAttnThreads = 256;                 // 16 half-warps
constexpr int kAttnHalfWarps = kAttnThreads / 16;
constexpr int kPartStride = kHeadDim + 2;         // o[128] (unnormalised), m, l per split

struct AttnParams {
  const __nv_bfloat16* q;   // [B][Hq][128]
  KvDev kv;
  const int* idx;           // [B][Hq][idx_stride] or nullptr = all positions [0, t)
  const int* count;         // [B][Hq] (ignored when idx == nullptr)
  int idx_stride;
  int num_q_heads, group_size;
  int splits;
  float* partials;          // [B][Hq][splits][kPartStride]
  unsigned int* tickets;    // [B][Hq], zero on entry, zero again on exit
  __nv_bfloat16* out;       // [B][Hq][128]
  float* out_lse;           // [B][Hq] or nullptr
  const float* lse_full;    // [B][Hq] or nullptr
  float* out_delta;         // [B][Hq] or nullptr: 1 - exp(lse - lse_full)
  uint32_t* flags;
};

// grid (splits, Hq, B).  Each half-warp owns blocks of 16 consecutive list entries; a lane
// holds 8 of the 128 elements of a row, so one 16-byte load per lane fetches a whole row
// per half-warp.  Four K rows and four V rows are in flight per half-warp.  Every
// half-warp keeps its own online-softmax state (log2 domain); states are combined in shared
// memory, written as a split partial, and the last CTA to arrive for a (b, h) merges the
// splits (ticket counter, no waiting).
__global__ void __launch_bounds__(kAttnThreads) gather_attn_kernel(AttnParams p) {
  const int split = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
  const int unit = b * p.num_q_heads + h;
  const int kvh = h / p.group_size;
  const int tid = threadIdx.x, l16 = tid & 15, hw = tid >> 4;
  const int t = __ldg(p.kv.seq_lens + b);
  const int cnt = p.idx ? min(__ldg(p.count + unit), p.idx_stride) : t;
  int per = (cnt + p.splits - 1) / p.splits;
  per = (per + 15) & ~15;
  const int start = min(split * per, cnt);
  const int end = min(start + per, cnt);
  const int* list = p.idx ? p.idx + (long long)unit * p.idx_stride : nullptr;

  float qf[8];
  {
    const uint4 x = *reinterpret_cast<const uint4*>(p.q + (long long)unit * kHeadDim + l16 * 8);
    const float c = kScale * kLog2e;   // logits are kept in the log2 domain
    qf[0] = bf_lo(x.x) * c; qf[1] = bf_hi(x.x) * c; qf[2] = bf_lo(x.y) * c; qf[3] = bf_hi(x.y) * c;
    qf[4] = bf_lo(x.z) * c; qf[5] = bf_hi(x.z) * c; qf[6] = bf_lo(x.w) * c; qf[7] = bf_hi(x.w) * c;
  }
  float m = -INFINITY, l = 0.f;
  float o[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) o[i] = 0.f;

  // the trip count is uniform over a warp (its two half-warps take adjacent 16-entry blocks)
  for (int jw = start + (tid >> 5) * 32; jw < end; jw += kAttnHalfWarps * 16) {
    const int j0 = jw + (hw & 1) * 16;
    int my = -1;
    if (j0 + l16 < end) {
      my = list ? __ldg(list + j0 + l16) : j0 + l16;
      if ((unsigned)my >= (unsigned)t) {
        atomicOr(p.flags, kFlagBadIndex);
        my = -1;
      }
    }
#pragma unroll
    for (int e0 = 0; e0 < 16; e0 += 4) {
      uint4 kx[4], vx[4];
      bool ok[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int pos = __shfl_sync(0xffffffffu, my, e0 + u, 16);
        ok[u] = pos >= 0;
        kx[u] = make_uint4(0u, 0u, 0u, 0u);
        vx[u] = make_uint4(0u, 0u, 0u, 0u);
        if (ok[u]) {
          const long long off = row_offset(p.kv, b, kvh, pos, p.flags);
          if (off >= 0) {
            kx[u] = ldg_stream(p.kv.k + off + l16 * 8);
            vx[u] = ldg_stream(p.kv.v + off + l16 * 8);
          } else {
            ok[u] = false;
          }
        }
      }
      float s[4];
      float mn = m;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        s[u] = half_warp_sum(dot8(kx[u], qf));
        if (!ok[u]) s[u] = -INFINITY;
        mn = fmaxf(mn, s[u]);
      }
      if (mn != -INFINITY) {
        const float corr = exp2f(m - mn);
        l *= corr;
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] *= corr;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const float pw = exp2f(s[u] - mn);
          l += pw;
          o[0] = fmaf(pw, bf_lo(vx[u].x), o[0]); o[1] = fmaf(pw, bf_hi(vx[u].x), o[1]);
          o[2] = fmaf(pw, bf_lo(vx[u].y), o[2]); o[3] = fmaf(pw, bf_hi(vx[u].y), o[3]);
          o[4] = fmaf(pw, bf_lo(vx[u].z), o[4]); o[5] = fmaf(pw, bf_hi(vx[u].z), o[5]);
          o[6] = fmaf(pw, bf_lo(vx[u].w), o[6]); o[7] = fmaf(pw, bf_hi(vx[u].w), o[7]);
        }
        m = mn;
      }
    }
  }

  // ---- combine the 16 half-warp states of this CTA
  __shared__ float sm_o[kAttnHalfWarps][kHeadDim];
  __shared__ float sm_m[kAttnHalfWarps], sm_l[kAttnHalfWarps];
  __shared__ bool is_last;
#pragma unroll
  for (int i = 0; i < 8; ++i) sm_o[hw][l16 * 8 + i] = o[i];
  if (l16 == 0) { sm_m[hw] = m; sm_l[hw] = l; }
  __syncthreads();
  float* part = p.partials + ((long long)unit * p.splits + split) * kPartStride;
  if (tid < kHeadDim) {
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kAttnHalfWarps; ++w) M = fmaxf(M, sm_m[w]);
    float acc = 0.f, L = 0.f;
    if (M != -INFINITY) {
#pragma unroll
      for (int w = 0; w < kAttnHalfWarps; ++w) {
        const float sc = exp2f(sm_m[w] - M);
        acc = fmaf(sm_o[w][tid], sc, acc);
        L = fmaf(sm_l[w], sc, L);
      }
    }
    if (p.splits == 1) {
      // single split: finish here
      p.out[(long long)unit * kHeadDim + tid] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
      if (tid == 0) {
        const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
        if (p.out_lse) p.out_lse[unit] = lse;
        if (p.out_delta) p.out_delta[unit] = L > 0.f ? -expm1f(lse - p.lse_full[unit]) : 1.f;
      }
    } else {
      part[tid] = acc;
      if (tid == 0) { part[kHeadDim] = M; part[kHeadDim + 1] = L; }
    }
  }
  if (p.splits == 1) return;

  // ---- the last CTA of this (b, h) merges the split partials
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned int ticket = atomicAdd(p.tickets + unit, 1u);
    is_last = (ticket == (unsigned int)p.splits - 1u);
    if (is_last) p.tickets[unit] = 0u;   // ready for the next launch
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  if (tid < kHeadDim) {
    const float* base = p.partials + (long long)unit * p.splits * kPartStride;
    float M = -INFINITY;
    for (int s = 0; s < p.splits; ++s) M = fmaxf(M, __ldcg(base + s * kPartStride + kHeadDim));
    float acc = 0.f, L = 0.f;
    if (M != -INFINITY) {
      for (int s = 0; s < p.splits; ++s) {
        const float sc = exp2f(__ldcg(base + s * kPartStride + kHeadDim) - M);
        acc = fmaf(__ldcg(base + s * kPartStride + tid), sc, acc);
        L = fmaf(__ldcg(base + s * kPartStride + kHeadDim + 1), sc, L);
      }
    }
    p.out[(long long)unit * kHeadDim + tid] = __float2bfloat16_rn(L > 0.f ? acc / L : 0.f);
    if (tid == 0) {
      const float lse = L > 0.f ? (M + log2f(L)) * kLn2 : -INFINITY;
      if (p.out_lse) p.out_lse[unit] = lse;
      if (p.out_delta) p.out_delta[unit] = L > 0.f ? -expm1f(lse - p.lse_full[unit]) : 1.f;
    }
  }
}

// delta = 1 - exp(lse_C - lse_full)  (Sec. 2.3), one thread per (b, h).
__global__ void delta_kernel(const float* __restrict__ lse_c, const float* __restrict__ lse_full,
                             float* __restrict__ out, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = (lse_c[i] == -INFINITY) ? 1.f : -expm1f(lse_c[i] - lse_full[i]);
}

// Reduce the scoring pass' per-chunk (m, l) partials to lse_full (used when no selection runs).
__global__ void lse_reduce_kernel(const float2* __restrict__ part_ml, int nchunks,
                                  float* __restrict__ lse_full, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float mm = -INFINITY, ll = 0.f;
  for (int c = 0; c < nchunks; ++c) {
    const float2 x = part_ml[(long long)i * nchunks + c];
    ml_combine(mm, ll, x.x, x.y);
  }
  lse_full[i] = ll > 0.f ? (mm + log2f(ll)) * kLn2 : -INFINITY;
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
