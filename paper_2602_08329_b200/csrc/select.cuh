// Retrieval pass, part 2: exact top-k over the middle range (Sec. 4.1 "Selection
// Criteria"), descending-logit order with ties broken by lower position, then the
// neighbour dilation of Eq. 10.  One CTA per (sequence, query head).
//
// Fast path: a 1-in-16 sample of the unit's logits is histogrammed on the top 11 bits of the
// order-preserving key; from it a conservative bin d_lo is chosen so that, with a wide
// margin, at least k logits lie in bins >= d_lo.  ONE pass over all logits then collects those
// into a short list in shared memory (about 1.5-2 k entries), and everything else -- the exact
// bin of the k-th key, the remaining 21 key bits, ties -- is resolved on that list.  Small
// problems (at most 8192 candidates) skip the sample and list every candidate.  If the list
// comes out too short or too long (sampling bad luck, or degenerate inputs such as all-equal
// logits), a generic 4 x 8-bit radix select over the logits in global memory takes over; it
// orders ties by position explicitly.
#pragma once
#include "common.cuh"

namespace prhs {

constexpr int kSelThreads = 512;
constexpr int kHistBits = 11;
constexpr int kHistBins = 1 << kHistBits;          // 2048
constexpr int kHistShift = 32 - kHistBits;         // key >> 21
constexpr int kSelMiscWords = 64;
constexpr int kCandCap = 8192;                      // candidate list entries (8 bytes each)
constexpr int kSampleStride = 16;

struct SelectParams {
  const float* scores;      // [B][Hq][ld]
  int ld;
  const float2* part_ml;    // [B][Hq][nchunks] (m, l) in the log2 domain; chunks past t are unset
  int nchunks, chunk_rows;
  const int* seq_lens;
  const int* k_per_seq;     // or nullptr
  int k, sinks, window, r, m;
  double psaw_c;            // sliding-window factor of this layer (0 = off)
  int max_k, shat_cap, num_q_heads;
  int* sstar_desc;          // [B][Hq][slots][max_k]
  int* sstar_asc;           // [B][Hq][slots][max_k]
  int* shat_asc;            // [B][Hq][slots][shat_cap]
  int* n_star;              // [B][Hq][slots]
  int* n_hat;               // [B][Hq][slots]
  const int* need;          // [B][Hq] or nullptr: only units with need != 0 select (cosine gate)
  const int* slot_of;       // [B][Hq] or nullptr (slot 0): where the new set goes
  int slots;
  int* anchor_t;            // [B]: t_b at this retrieval
  int* out_idx;             // optional [B][Hq][max_k]
  int* out_count;           // optional
  float* lse_full;          // [B][Hq] workspace
  float* out_lse_full;      // optional
  uint32_t* flags;
  int sort_cap;             // power of two >= max_k
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

// Append `v` to list[] for the lanes with f set: one shared-memory atomic per warp.
__device__ __forceinline__ void warp_append(bool f, unsigned long long v, unsigned long long* list,
                                            uint32_t* counter, uint32_t cap) {
  const uint32_t bal = __ballot_sync(0xffffffffu, f);
  if (bal == 0u) return;
  const int lane = threadIdx.x & 31;
  uint32_t base = 0u;
  if (lane == (__ffs(bal) - 1)) base = atomicAdd(counter, (uint32_t)__popc(bal));
  base = __shfl_sync(0xffffffffu, base, __ffs(bal) - 1);
  const uint32_t slot = base + __popc(bal & ((1u << lane) - 1u));
  if (f && slot < cap) list[slot] = v;
}

__device__ __forceinline__ unsigned long long make_entry(uint32_t key, int pos) {
  return ((unsigned long long)key << 32) | (unsigned long long)(0xffffffffu - (uint32_t)pos);
}

// Digit bin that holds the rem-th largest element, scanning bins from the top.
// hist has nb bins (nb a multiple of 32, nb / 32 <= 64 bins per lane).  Warp 0 only.
// Writes misc[0] = bin, misc[1] = how many of that bin are still needed, misc[2] = its count.
__device__ __forceinline__ void find_bin_from_top(const uint32_t* hist, int nb, int rem, uint32_t* misc) {
  const int lane = threadIdx.x & 31;
  const int per = nb >> 5;
  int s = 0;   // lane's bins are read in a rotated order: per is a multiple of 32 for large nb
  for (int j = 0; j < per; ++j) s += (int)hist[lane * per + ((j + lane) % per)];
  int incl = s;   // sum over lanes >= lane
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int x = __shfl_down_sync(0xffffffffu, incl, off);
    if (lane + off < 32) incl += x;
  }
  const int above = incl - s;
  if (above < rem && rem <= incl) {
    int c = above;
    for (int j = per - 1; j >= 0; --j) {
      const int hc = (int)hist[lane * per + j];
      if (c + hc >= rem) {
        misc[0] = (uint32_t)(lane * per + j);
        misc[1] = (uint32_t)(rem - c);
        misc[2] = (uint32_t)hc;
        break;
      }
      c += hc;
    }
  }
}

// ---- block-wide bitonic sort, descending, of P (a power of two >= 64) 64-bit entries in
// shared memory.  Compare-exchange steps with a stride below 64 stay inside one 64-entry
// block, which a warp holds in registers (two entries per lane) and resolves with shuffles;
// only strides >= 64 go through shared memory with a CTA barrier.  All threads call it.
__device__ __forceinline__ void warp_sort_steps(unsigned long long& a, unsigned long long& b, int pos_a,
                                                int size, int first_stride) {
  const int lane = threadIdx.x & 31;
  const int pos_b = pos_a + 32;
  for (int stride = first_stride; stride > 0; stride >>= 1) {
    if (stride == 32) {
      const bool desc = (pos_a & size) == 0;
      if ((a < b) == desc) { const unsigned long long x = a; a = b; b = x; }
    } else {
      const unsigned long long oa = __shfl_xor_sync(0xffffffffu, a, stride);
      const unsigned long long ob = __shfl_xor_sync(0xffffffffu, b, stride);
      const bool lower = (lane & stride) == 0;
      const bool da = (pos_a & size) == 0, db = (pos_b & size) == 0;
      a = (lower == da) ? (a > oa ? a : oa) : (a < oa ? a : oa);
      b = (lower == db) ? (b > ob ? b : ob) : (b < ob ? b : ob);
    }
  }
}

__device__ __forceinline__ void block_sort_desc(unsigned long long* buf, int P) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nwarps = blockDim.x >> 5;
  const int nblocks = P >> 6;
  // sizes 2 .. 64: entirely inside 64-entry blocks
  for (int blk = warp; blk < nblocks; blk += nwarps) {
    const int pos_a = blk * 64 + lane;
    unsigned long long a = buf[pos_a], b = buf[pos_a + 32];
    for (int size = 2; size <= 64; size <<= 1) warp_sort_steps(a, b, pos_a, size, size >> 1);
    buf[pos_a] = a;
    buf[pos_a + 32] = b;
  }
  __syncthreads();
  for (int size = 128; size <= P; size <<= 1) {
    for (int stride = size >> 1; stride >= 64; stride >>= 1) {
      for (int x = tid; x < (P >> 1); x += blockDim.x) {
        const int i = 2 * x - (x & (stride - 1));
        const int j = i + stride;
        const bool desc = ((i & size) == 0);
        const unsigned long long a = buf[i], c = buf[j];
        if ((a < c) == desc) { buf[i] = c; buf[j] = a; }
      }
      __syncthreads();
    }
    for (int blk = warp; blk < nblocks; blk += nwarps) {
      const int pos_a = blk * 64 + lane;
      unsigned long long a = buf[pos_a], b = buf[pos_a + 32];
      warp_sort_steps(a, b, pos_a, size, 32);
      buf[pos_a] = a;
      buf[pos_a + 32] = b;
    }
    __syncthreads();
  }
}

__global__ void __launch_bounds__(kSelThreads, 2) select_kernel(SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw);                     // kHistBins
  uint32_t* misc = hist + kHistBins;                                          // kSelMiscWords
  unsigned long long* wbuf = reinterpret_cast<unsigned long long*>(misc + kSelMiscWords);  // sort_cap
  unsigned long long* cand = wbuf + p.sort_cap;                               // kCandCap
  uint32_t* bm = reinterpret_cast<uint32_t*>(cand);                           // bitmap aliases cand

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int unit = blockIdx.x;
  if (p.need != nullptr && __ldg(p.need + unit) == 0) return;     // this head shares: no retrieval
  const long long sunit = (long long)unit * p.slots + (p.slot_of ? __ldg(p.slot_of + unit) : 0);
  const int b = unit / p.num_q_heads;
  const int t = __ldg(p.seq_lens + b);
  int k = p.k_per_seq ? __ldg(p.k_per_seq + b) : p.k;
  k = max(0, min(k, p.max_k));
  const int lo = max(min(p.sinks, t), psaw_start(p.psaw_c, t));   // first middle candidate
  const int n = max(t - p.window - lo, 0);
  const int kk = min(k, n);
  const int m_eff = min(p.m < 0 ? k / 3 : p.m, kk);
  const float* g = p.scores + (long long)unit * p.ld + lo;

  // full-softmax log-sum-exp from the scoring pass' per-chunk partials
  if (warp == 1) {
    float mm = -INFINITY, ll = 0.f;
    const int nch = p.chunk_rows > 0 ? min(p.nchunks, (t + p.chunk_rows - 1) / p.chunk_rows) : p.nchunks;
    for (int c = lane; c < nch; c += 32) {
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
  if (tid == 0) {
    if ((unit % p.num_q_heads) == 0) p.anchor_t[b] = t;
    misc[4] = 0u;   // winners appended
    misc[5] = 0u;   // candidates appended
  }
  __syncthreads();

  int total = 0;          // entries in wbuf to sort; the first kk after sorting are S*
  bool fast_ok = false;
  if (kk > 0) {
    // ---------------- fast path
    // 1. conservative bin d_lo from a sample (or 0: list everything)
    uint32_t d_lo = 0u;
    if (n > kCandCap) {
      for (int i = tid; i < kHistBins; i += kSelThreads) hist[i] = 0u;
      __syncthreads();
      const int ns = n / kSampleStride;
      for (int j0 = 0; j0 < ns; j0 += 8 * kSelThreads) {     // 8 independent loads in flight
        uint32_t u8[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const int j = j0 + x * kSelThreads + tid;
          u8[x] = j < ns ? float_to_key(__ldcg(g + j * kSampleStride + (j & (kSampleStride - 1)))) : 0u;
        }
#pragma unroll
        for (int x = 0; x < 8; ++x)
          if (j0 + x * kSelThreads + tid < ns) atomicAdd(&hist[u8[x] >> kHistShift], 1u);
      }
      __syncthreads();
      // want at least 1.5 k/16 + 16 sampled logits at or above d_lo (several sigma of margin)
      const int want = min(ns, (3 * kk) / (2 * kSampleStride) + 16);
      if (warp == 0) find_bin_from_top(hist, kHistBins, want, misc);
      __syncthreads();
      d_lo = misc[0];
      __syncthreads();
    }
    // 2. one pass over the logits: 16 independent loads in flight per thread, then one warp
    //    scan and one shared-memory atomic per warp and batch to place the listed entries
    const int nrounds = (n + kSelThreads - 1) / kSelThreads;
    for (int rd0 = 0; rd0 < nrounds; rd0 += 16) {
      uint32_t u16[16];
#pragma unroll
      for (int x = 0; x < 16; ++x) {
        const int i = (rd0 + x) * kSelThreads + tid;
        u16[x] = i < n ? float_to_key(__ldcg(g + i)) : 0u;
      }
      uint32_t cmask = 0u;
#pragma unroll
      for (int x = 0; x < 16; ++x) {
        const int i = (rd0 + x) * kSelThreads + tid;
        cmask |= (uint32_t)(i < n && (u16[x] >> kHistShift) >= d_lo) << x;
      }
      const uint32_t mine = (uint32_t)__popc(cmask);
      uint32_t incl = mine;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const uint32_t x = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += x;
      }
      uint32_t bc = 0u;
      if (lane == 31 && incl) bc = atomicAdd(&misc[5], incl);
      uint32_t oc = __shfl_sync(0xffffffffu, bc, 31) + incl - mine;
#pragma unroll
      for (int x = 0; x < 16; ++x) {
        if ((cmask >> x) & 1u) {
          if (oc < (uint32_t)kCandCap) cand[oc] = make_entry(u16[x], lo + (rd0 + x) * kSelThreads + tid);
          ++oc;
        }
      }
    }
    __syncthreads();
    const int ncand = (int)misc[5];
    fast_ok = ncand >= kk && ncand <= kCandCap;
    if (fast_ok) {
      // 3. exact histogram of the list -> bin d1 of the kk-th largest key
      for (int i = tid; i < kHistBins; i += kSelThreads) hist[i] = 0u;
      __syncthreads();
      for (int i = tid; i < ncand; i += kSelThreads)
        atomicAdd(&hist[(uint32_t)(cand[i] >> 32) >> kHistShift], 1u);
      __syncthreads();
      if (warp == 0) find_bin_from_top(hist, kHistBins, kk, misc);
      __syncthreads();
      uint32_t prefix = misc[0] << kHistShift;
      int rem = (int)misc[1], eq = (int)misc[2];
      __syncthreads();
      // 4. the remaining 21 key bits within that bin: 3 passes of 7 bits
      if (rem < eq) {
        for (int pass = 0; pass < 3; ++pass) {
          const int shift = kHistShift - 7 * (pass + 1);
          const uint32_t mask = 0xffffffffu << (shift + 7);
          if (tid < 128) hist[tid] = 0u;
          __syncthreads();
          for (int i = tid; i < ncand; i += kSelThreads) {
            const uint32_t u = (uint32_t)(cand[i] >> 32);
            if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 127u], 1u);
          }
          __syncthreads();
          if (warp == 0) find_bin_from_top(hist, 128, rem, misc);
          __syncthreads();
          prefix |= misc[0] << shift;
          rem = (int)misc[1];
          eq = (int)misc[2];
          __syncthreads();
        }
      }   // else every key of bin d1 is needed: the threshold is the start of the bin
      const uint32_t T = prefix;            // keys >= T: the winners plus the surplus ties at T
      // 5. winners and ties into the sort buffer; sorting orders ties by position and the
      //    surplus falls behind the first kk entries
      const int crounds = (ncand + kSelThreads - 1) / kSelThreads;
      for (int rd = 0; rd < crounds; ++rd) {
        const int i = rd * kSelThreads + tid;
        unsigned long long e = 0ull;
        if (i < ncand) e = cand[i];
        warp_append(i < ncand && (uint32_t)(e >> 32) >= T, e, wbuf, &misc[4], (uint32_t)p.sort_cap);
      }
      __syncthreads();
      total = (int)misc[4];
      if (total > p.sort_cap || total < kk) fast_ok = false;
    }
    __syncthreads();

    if (!fast_ok) {
      // ---------------- generic path: 4 x 8-bit radix select over the logits in global memory
      if (tid == 0) {
        atomicOr(p.flags, kFlagSelectFallback);
        misc[4] = 0u;
      }
      uint32_t prefix = 0u;
      int rem = kk, eq = 0;
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t mask = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        for (int i = tid; i < n; i += kSelThreads) {
          const uint32_t u = float_to_key(__ldcg(g + i));
          if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (warp == 0) find_bin_from_top(hist, 256, rem, misc);
        __syncthreads();
        prefix |= misc[0] << shift;
        rem = (int)misc[1];
        eq = (int)misc[2];
      }
      const uint32_t T = prefix;
      const int need = rem, gt_total = kk - need;
      const bool all_ties = (eq == need);
      const int nrounds2 = (n + kSelThreads - 1) / kSelThreads;
      for (int rd = 0; rd < nrounds2; ++rd) {
        const int i = rd * kSelThreads + tid;
        uint32_t u = 0u;
        if (i < n) u = float_to_key(__ldcg(g + i));
        warp_append(i < n && (u > T || (all_ties && u == T)), make_entry(u, lo + i), wbuf, &misc[4],
                    (uint32_t)p.sort_cap);
      }
      if (!all_ties) {
        // ties at T, lowest positions first
        int base = 0;
        for (int c0 = 0; c0 < n && base < need; c0 += kSelThreads) {
          const int i = c0 + tid;
          const bool f = (i < n) && float_to_key(__ldcg(g + i)) == T;
          const uint32_t bal = __ballot_sync(0xffffffffu, f);
          if (lane == 0) misc[8 + warp] = __popc(bal);
          __syncthreads();
          int before = 0, tot = 0;
          for (int w = 0; w < kSelThreads / 32; ++w) {
            const int c = (int)misc[8 + w];
            if (w < warp) before += c;
            tot += c;
          }
          const int rank = base + before + __popc(bal & ((1u << lane) - 1u));
          if (f && rank < need) wbuf[gt_total + rank] = make_entry(T, lo + i);
          base += tot;
          __syncthreads();
        }
      }
      total = kk;
      __syncthreads();
    }
  }

  // ---- sort: descending key, ascending position among equal keys
  int P = 64;
  while (P < total) P <<= 1;
  for (int i = total + tid; i < P; i += kSelThreads) wbuf[i] = 0ull;
  __syncthreads();
  block_sort_desc(wbuf, P);

  // ---- S* in descending-logit order
  int* sd = p.sstar_desc + sunit * p.max_k;
  for (int e = tid; e < p.max_k; e += kSelThreads) {
    const int v = e < kk ? (int)(0xffffffffu - (uint32_t)(wbuf[e] & 0xffffffffull)) : -1;
    sd[e] = v;
    if (p.out_idx) p.out_idx[(long long)unit * p.max_k + e] = v;
  }
  if (tid == 0) {
    p.n_star[sunit] = kk;
    if (p.out_count) p.out_count[unit] = kk;
  }

  // ---- ascending S*, then the dilated S^ (Eq. 10), through a position bitmap
  const int words = (t + 31) >> 5;
  for (int w = tid; w < words; w += kSelThreads) bm[w] = 0u;
  __syncthreads();
  for (int e = tid; e < kk; e += kSelThreads) {
    const uint32_t pos = 0xffffffffu - (uint32_t)(wbuf[e] & 0xffffffffull);
    atomicOr(&bm[pos >> 5], 1u << (pos & 31u));
  }
  __syncthreads();
  compact_bitmap(bm, words, p.sstar_asc + sunit * p.max_k, p.max_k, misc + 8);
  __syncthreads();   // every thread has finished reading the bitmap before it grows
  for (int e = tid; e < m_eff; e += kSelThreads) {
    const int pos = (int)(0xffffffffu - (uint32_t)(wbuf[e] & 0xffffffffull));
    for (int j = -p.r; j <= p.r; ++j) {
      const int x = pos + j;
      if (x >= 0 && x < t) atomicOr(&bm[x >> 5], 1u << (x & 31));
    }
  }
  __syncthreads();
  const int nh = compact_bitmap(bm, words, p.shat_asc + sunit * p.shat_cap, p.shat_cap,
                                misc + 8);
  if (tid == 0) p.n_hat[sunit] = min(nh, p.shat_cap);
}

}  // namespace prhs
