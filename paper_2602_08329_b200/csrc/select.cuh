// Retrieval pass, part 2: exact top-k over the middle range (Sec. 4.1 "Selection
// Criteria"), descending-logit order with ties broken by lower position, then the
// neighbour dilation of Eq. 10.  One CTA per (sequence, query head).
#pragma once
#include "common.cuh"

namespace prhs {

constexpr int kSelThreads = 1024;
constexpr int kSelHeaderWords = 256 + 64;   // radix histogram + scalars/scan scratch

struct SelectParams {
  const float* scores;      // [B][Hq][ld]
  int ld;
  const float2* part_ml;    // [B][Hq][nchunks] (m, l) in the log2 domain
  int nchunks;
  const int* seq_lens;
  const int* k_per_seq;     // or nullptr
  int k, sinks, window, r, m;
  int max_k, shat_cap, num_q_heads;
  int* sstar_desc;          // [B][Hq][max_k]
  int* sstar_asc;           // [B][Hq][max_k]
  int* shat_asc;            // [B][Hq][shat_cap]
  int* n_star;              // [B][Hq]
  int* n_hat;               // [B][Hq]
  int* anchor_t;            // [B]: t_b at this retrieval
  int* out_idx;             // optional [B][Hq][max_k]
  int* out_count;           // optional
  float* lse_full;          // [B][Hq] workspace
  float* out_lse_full;      // optional
  uint32_t* flags;
  int sort_cap;             // power of two >= max_k
  int resident_cap;         // candidates that fit in shared memory as keys
};

// Exclusive block scan of one int per thread; returns the exclusive prefix, *total gets the sum.
__device__ __forceinline__ int block_exclusive_scan(int v, uint32_t* ws /*>= 34 words*/, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int x = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += x;
  }
  if (lane == 31) ws[warp] = (uint32_t)incl;
  __syncthreads();
  if (warp == 0) {
    const int wt = (lane < (int)(blockDim.x >> 5)) ? (int)ws[lane] : 0;
    int wi = wt;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int x = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += x;
    }
    ws[lane] = (uint32_t)(wi - wt);
    if (lane == 31) ws[32] = (uint32_t)wi;
  }
  __syncthreads();
  const int res = incl - v + (int)ws[warp];
  *total = (int)ws[32];
  __syncthreads();
  return res;
}

// Ascending list of the set bits of bm[0..words): out[0..min(total,cap)); returns total.
__device__ __forceinline__ int compact_bitmap(const uint32_t* bm, int words, int* out, int cap,
                                              uint32_t* ws) {
  const int per = (words + (int)blockDim.x - 1) / (int)blockDim.x;
  const int w0 = min((int)threadIdx.x * per, words);
  const int w1 = min(w0 + per, words);
  int cnt = 0;
  for (int w = w0; w < w1; ++w) cnt += __popc(bm[w]);
  int total;
  int o = block_exclusive_scan(cnt, ws, &total);
  for (int w = w0; w < w1; ++w) {
    uint32_t x = bm[w];
    while (x) {
      const int bit = __ffs(x) - 1;
      if (o < cap) out[o] = w * 32 + bit;
      ++o;
      x &= x - 1;
    }
  }
  return total;
}

__global__ void __launch_bounds__(kSelThreads, 1) select_kernel(SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw);
  uint32_t* misc = hist + 256;
  unsigned long long* wbuf = reinterpret_cast<unsigned long long*>(misc + 64);
  uint32_t* region = reinterpret_cast<uint32_t*>(wbuf + p.sort_cap);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.x;
  const int b = unit / p.num_q_heads;
  const int t = __ldg(p.seq_lens + b);
  int k = p.k_per_seq ? __ldg(p.k_per_seq + b) : p.k;
  k = max(0, min(k, p.max_k));
  const int lo = min(p.sinks, t);
  const int n = max(t - p.window - lo, 0);
  const int kk = min(k, n);
  const int m_eff = min(p.m < 0 ? k / 3 : p.m, kk);

  // full-softmax log-sum-exp from the scoring pass' per-chunk partials
  if (warp == 0) {
    float mm = -INFINITY, ll = 0.f;
    for (int c = lane; c < p.nchunks; c += 32) {
      const float2 x = p.part_ml[(long long)unit * p.nchunks + c];
      ml_combine(mm, ll, x.x, x.y);
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, mm, off);
      const float l2 = __shfl_xor_sync(0xffffffffu, ll, off);
      ml_combine(mm, ll, m2, l2);
    }
    if (lane == 0) {
      const float lse = (ll > 0.f) ? (mm + log2f(ll)) * kLn2 : -INFINITY;
      p.lse_full[unit] = lse;
      if (p.out_lse_full) p.out_lse_full[unit] = lse;
    }
  }
  if (tid == 0 && (unit % p.num_q_heads) == 0) p.anchor_t[b] = t;

  const float* g = p.scores + (long long)unit * p.ld + lo;
  const bool resident = n <= p.resident_cap;
  if (resident) {
    for (int i = tid; i < n; i += kSelThreads) region[i] = float_to_key(__ldcg(g + i));
  } else if (tid == 0 && n > 0) {
    atomicOr(p.flags, kFlagSelectFallback);
  }
  if (tid == 0) misc[4] = 0u;
  __syncthreads();
  auto key_at = [&](int i) -> uint32_t {
    return resident ? region[i] : float_to_key(__ldcg(g + i));
  };

  // ---- radix select: the kk-th largest key T, and how many keys equal to T are needed
  uint32_t T = 0u;
  int need = 0, eq = 0;
  if (kk > 0) {
    int rem = kk;
    uint32_t prefix = 0u;
    for (int pass = 0; pass < 4; ++pass) {
      const int shift = 24 - 8 * pass;
      const uint32_t mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
      if (tid < 256) hist[tid] = 0u;
      __syncthreads();
      for (int i = tid; i < n; i += kSelThreads) {
        const uint32_t u = key_at(i);
        if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (warp == 0) {
        int s = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) s += (int)hist[lane * 8 + j];
        int incl = s;   // sum over lanes >= lane
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
          const int x = __shfl_down_sync(0xffffffffu, incl, off);
          if (lane + off < 32) incl += x;
        }
        const int above = incl - s;
        if (above < rem && rem <= incl) {
          int c = above;
          for (int j = 7; j >= 0; --j) {
            const int hc = (int)hist[lane * 8 + j];
            if (c + hc >= rem) {
              misc[0] = (uint32_t)(lane * 8 + j);
              misc[1] = (uint32_t)(rem - c);
              misc[2] = (uint32_t)hc;
              break;
            }
            c += hc;
          }
        }
      }
      __syncthreads();
      prefix |= misc[0] << shift;
      rem = (int)misc[1];
      eq = (int)misc[2];
    }
    T = prefix;
    need = rem;
  }

  // ---- collect the winners as (key << 32 | ~position): keys above T, then ties in position order
  const int gt_total = kk - need;
  if (kk > 0) {
    const bool all_ties = (eq == need);
    for (int i = tid; i < n; i += kSelThreads) {
      const uint32_t u = key_at(i);
      if (u > T || (all_ties && u == T)) {
        const uint32_t slot = atomicAdd(&misc[4], 1u);
        if (slot < (uint32_t)p.sort_cap)
          wbuf[slot] = ((unsigned long long)u << 32) | (unsigned long long)(0xffffffffu - (uint32_t)(lo + i));
      }
    }
    if (!all_ties) {
      int base = 0;
      for (int c0 = 0; c0 < n && base < need; c0 += kSelThreads) {
        const int i = c0 + tid;
        const bool f = (i < n) && key_at(i) == T;
        const uint32_t bal = __ballot_sync(0xffffffffu, f);
        if (lane == 0) misc[8 + warp] = __popc(bal);
        __syncthreads();
        int before = 0, total = 0;
        for (int w = 0; w < kSelThreads / 32; ++w) {
          const int c = (int)misc[8 + w];
          if (w < warp) before += c;
          total += c;
        }
        const int rank = base + before + __popc(bal & ((1u << lane) - 1u));
        if (f && rank < need)
          wbuf[gt_total + rank] =
              ((unsigned long long)T << 32) | (unsigned long long)(0xffffffffu - (uint32_t)(lo + i));
        base += total;
        __syncthreads();
      }
    }
  }
  // ---- sort the winners: descending key, ascending position among equal keys
  int P = 2;
  while (P < kk) P <<= 1;
  __syncthreads();
  for (int i = kk + tid; i < P; i += kSelThreads) wbuf[i] = 0ull;
  for (int size = 2; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      __syncthreads();
      for (int x = tid; x < (P >> 1); x += kSelThreads) {
        const int i = 2 * x - (x & (stride - 1));
        const int j = i + stride;
        const bool desc = ((i & size) == 0);
        const unsigned long long a = wbuf[i], c = wbuf[j];
        if ((a < c) == desc) { wbuf[i] = c; wbuf[j] = a; }
      }
    }
  }
  __syncthreads();

  // ---- S* in descending-logit order
  int* sd = p.sstar_desc + (long long)unit * p.max_k;
  for (int e = tid; e < p.max_k; e += kSelThreads) {
    const int v = e < kk ? (int)(0xffffffffu - (uint32_t)(wbuf[e] & 0xffffffffull)) : -1;
    sd[e] = v;
    if (p.out_idx) p.out_idx[(long long)unit * p.max_k + e] = v;
  }
  if (tid == 0) {
    p.n_star[unit] = kk;
    if (p.out_count) p.out_count[unit] = kk;
  }

  // ---- ascending S*, then the dilated S^ (Eq. 10), through a position bitmap
  uint32_t* bm = region;   // the keys are dead from here on
  const int words = (t + 31) >> 5;
  for (int w = tid; w < words; w += kSelThreads) bm[w] = 0u;
  __syncthreads();
  for (int e = tid; e < kk; e += kSelThreads) {
    const uint32_t pos = 0xffffffffu - (uint32_t)(wbuf[e] & 0xffffffffull);
    atomicOr(&bm[pos >> 5], 1u << (pos & 31u));
  }
  __syncthreads();
  compact_bitmap(bm, words, p.sstar_asc + (long long)unit * p.max_k, p.max_k, misc + 8);
  __syncthreads();   // every thread has finished reading the bitmap before it grows
  for (int e = tid; e < m_eff; e += kSelThreads) {
    const int pos = (int)(0xffffffffu - (uint32_t)(wbuf[e] & 0xffffffffull));
    for (int j = -p.r; j <= p.r; ++j) {
      const int x = pos + j;
      if (x >= 0 && x < t) atomicOr(&bm[x >> 5], 1u << (x & 31));
    }
  }
  __syncthreads();
  const int nh = compact_bitmap(bm, words, p.shat_asc + (long long)unit * p.shat_cap, p.shat_cap,
                                misc + 8);
  if (tid == 0) p.n_hat[unit] = min(nh, p.shat_cap);
}

}  // namespace prhs
