// Retrieval pass, part 2: exact top-k over the middle range (Sec. 4.1 "Selection
// Criteria"), descending-logit order with ties broken by lower position, then the
// neighbour dilation of Eq. 10.  One CTA per (sequence, query head); any multiple of 32 threads
// up to 1024 works; the library launches 512, or 256 / 1024 when that fills the SMs better.
//
// Fast path: every warp takes a stratified 1-in-16 sample of the unit's logits and finds by
// bisection on the top 13 key bits (a compare per sample and one warp reduction per bit) the
// value that a conservative share of them reach; the lower median over the warps is the
// threshold, chosen so that about 2 k logits pass it and, with a wide margin, no fewer than k.
// ONE pass over all logits (16-byte loads, one float compare each) lists the positions of those
// in shared memory, and everything else -- their keys, an exact 4 x 8-bit radix select of the
// k-th key, ties, the sort -- is resolved on that list, in place.  Small problems (no more
// candidates than the list holds) skip the sample and list every candidate.  If the list comes
// out too short or too long (sampling bad luck, or degenerate inputs such as all-equal logits),
// a generic 4 x 8-bit radix select over the logits in global memory takes over; it orders ties
// by position explicitly.  Logits crowd into a few histogram bins, so every histogram update
// first merges the lanes of a warp that hit the same bin (`match.any`) and issues one
// shared-memory atomic per distinct bin.  The winners are sorted by a merge sort (64-entry runs
// in registers, then one binary-search merge level per barrier).
#pragma once
#include "common.cuh"

namespace prhs {

constexpr int kSelMaxThreads = 512;
constexpr int kHistWords = 1024;                   // four 256-bin histograms
constexpr int kSelMiscWords = 128;
constexpr int kSampleStride = 16;

struct SelectParams {
  const float* scores;      // [B][Hq][ld], 16-byte aligned, ld a multiple of 4
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
  int sort_cap;             // power of two >= max_k: most entries the sort takes
  int cand_cap;             // candidate list entries (8 bytes each), >= sort_cap
  int two_bitmaps;          // room for two position bitmaps
  int unit_mul;             // 1, or the group size when one CTA selects for a whole KV group (its first head's rows)
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

// The same for two ints per thread at once (one set of barriers).  ws >= 68 words.
__device__ __forceinline__ void block_exclusive_scan2(int va, int vb, uint32_t* ws, int* ea, int* eb,
                                                      int* ta, int* tb) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int ia = va, ib = vb;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int xa = __shfl_up_sync(0xffffffffu, ia, off);
    const int xb = __shfl_up_sync(0xffffffffu, ib, off);
    if (lane >= off) { ia += xa; ib += xb; }
  }
  if (lane == 31) { ws[warp] = (uint32_t)ia; ws[34 + warp] = (uint32_t)ib; }
  __syncthreads();
  if (warp == 0) {
    const bool in = lane < (int)(blockDim.x >> 5);
    const int wa = in ? (int)ws[lane] : 0, wb = in ? (int)ws[34 + lane] : 0;
    int sa = wa, sb = wb;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int xa = __shfl_up_sync(0xffffffffu, sa, off);
      const int xb = __shfl_up_sync(0xffffffffu, sb, off);
      if (lane >= off) { sa += xa; sb += xb; }
    }
    ws[lane] = (uint32_t)(sa - wa);
    ws[34 + lane] = (uint32_t)(sb - wb);
    if (lane == 31) { ws[32] = (uint32_t)sa; ws[66] = (uint32_t)sb; }
  }
  __syncthreads();
  *ea = ia - va + (int)ws[warp];
  *eb = ib - vb + (int)ws[34 + warp];
  *ta = (int)ws[32];
  *tb = (int)ws[66];
  __syncthreads();
}

__device__ __forceinline__ int emit_bits(uint32_t x, int base, int* out, int o, int cap) {
  while (x) {
    const int bit = __ffs(x) - 1;
    if (o < cap) out[o] = base + bit;
    ++o;
    x &= x - 1;
  }
  return o;
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
  for (int w = w0; w < w1; ++w) o = emit_bits(bm[w], w * 32, out, o, cap);
  return total;
}

// Two bitmaps of the same length listed in one sweep (one scan, one set of barriers).
__device__ __forceinline__ void compact_two(const uint32_t* bma, const uint32_t* bmb, int words, int* outa,
                                            int capa, int* outb, int capb, uint32_t* ws, int* ta, int* tb) {
  const int per = (words + (int)blockDim.x - 1) / (int)blockDim.x;
  const int w0 = min((int)threadIdx.x * per, words);
  const int w1 = min(w0 + per, words);
  int ca = 0, cb = 0;
  for (int w = w0; w < w1; ++w) {
    ca += __popc(bma[w]);
    cb += __popc(bmb[w]);
  }
  int oa, ob;
  block_exclusive_scan2(ca, cb, ws, &oa, &ob, ta, tb);
  for (int w = w0; w < w1; ++w) {
    oa = emit_bits(bma[w], w * 32, outa, oa, capa);
    ob = emit_bits(bmb[w], w * 32, outb, ob, capb);
  }
}

// hist[bin] += 1 for the lanes with `valid`, one atomic per distinct bin of the warp.  Every lane
// of the warp must call it.
__device__ __forceinline__ void hist_add(uint32_t* hist, uint32_t bin, bool valid) {
  const uint32_t peers = __match_any_sync(0xffffffffu, valid ? bin : 0xffffffffu);
  if (valid && (int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
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

// The warp's sample of logits -- NSEC aligned 32-byte sectors (8 logits each) per lane: sample
// x * nt + slot of S, one sector out of every sec_stride -- and the largest value, at the
// resolution of the top 13 key bits, that at least rw of them reach.  Whole sectors, because the
// logits of a long context do not all stay in L2 and DRAM serves a scattered 4-byte read at
// the price of a sector.  Bisection on the key bits; the count is a compare per sample and one
// warp reduction per bit.
constexpr int kThrBits = 13;
template <int NSEC>
__device__ __forceinline__ uint32_t sample_quantile(const float* gal, int S, int sec_stride, int nt, int slot, int rw) {
  uint32_t u[8 * NSEC];
#pragma unroll
  for (int x = 0; x < NSEC; ++x) {
    const int sidx = x * nt + slot;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
    const bool ok = sidx < S;
    if (ok) {
      const float4* src = reinterpret_cast<const float4*>(gal + ((long long)sidx * sec_stride + ((sidx * 5) & 15)) * 8);
      a = __ldcg(src);
      b = __ldcg(src + 1);
    }
    u[8 * x + 0] = ok ? float_to_key(a.x) : 0u;
    u[8 * x + 1] = ok ? float_to_key(a.y) : 0u;
    u[8 * x + 2] = ok ? float_to_key(a.z) : 0u;
    u[8 * x + 3] = ok ? float_to_key(a.w) : 0u;
    u[8 * x + 4] = ok ? float_to_key(b.x) : 0u;
    u[8 * x + 5] = ok ? float_to_key(b.y) : 0u;
    u[8 * x + 6] = ok ? float_to_key(b.z) : 0u;
    u[8 * x + 7] = ok ? float_to_key(b.w) : 0u;
  }
  uint32_t prefix = 0u;
#pragma unroll 1
  for (int bit = 31; bit > 31 - kThrBits; --bit) {
    const uint32_t trial = prefix | (1u << bit);
    int cnt = 0;
#pragma unroll
    for (int x = 0; x < 8 * NSEC; ++x) cnt += u[x] >= trial ? 1 : 0;
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (cnt >= rw) prefix = trial;
  }
  return prefix;
}

// The same for a short range (at most one sampled sector per two lanes): the two lanes of a pair
// take one half of a sector each, so that every lane of the warp holds four logits.
__device__ __forceinline__ uint32_t sample_quantile_half(const float* gal, int S, int sec_stride, int nw, int rw) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int sidx = (lane >> 1) * nw + warp;
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
  const bool ok = sidx < S;
  if (ok) a = __ldcg(reinterpret_cast<const float4*>(gal + ((long long)sidx * sec_stride + ((sidx * 5) & 15)) * 8) + (lane & 1));
  const uint32_t u0 = ok ? float_to_key(a.x) : 0u, u1 = ok ? float_to_key(a.y) : 0u;
  const uint32_t u2 = ok ? float_to_key(a.z) : 0u, u3 = ok ? float_to_key(a.w) : 0u;
  uint32_t prefix = 0u;
#pragma unroll 1
  for (int bit = 31; bit > 31 - kThrBits; --bit) {
    const uint32_t trial = prefix | (1u << bit);
    int cnt = (u0 >= trial ? 1 : 0) + (u1 >= trial ? 1 : 0) + (u2 >= trial ? 1 : 0) + (u3 >= trial ? 1 : 0);
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    if (cnt >= rw) prefix = trial;
  }
  return prefix;
}

// Warp-wide: the digit (of 256 bins, h 16-byte aligned) that holds the rem-th largest entry counted
// from the top bin; every lane receives the bin, how many of that bin are still needed, and the
// bin's count.
__device__ __forceinline__ void find_bin_warp256(const uint32_t* h, int rem, int* bin, int* rem_out, int* eq_out) {
  const int lane = threadIdx.x & 31;
  const uint4 lo4 = *reinterpret_cast<const uint4*>(h + lane * 8);
  const uint4 hi4 = *reinterpret_cast<const uint4*>(h + lane * 8 + 4);
  const int c[8] = {(int)lo4.x, (int)lo4.y, (int)lo4.z, (int)lo4.w, (int)hi4.x, (int)hi4.y, (int)hi4.z, (int)hi4.w};
  int s = 0;
#pragma unroll
  for (int j = 0; j < 8; ++j) s += c[j];
  int incl = s;     // sum over lanes >= lane
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int x = __shfl_down_sync(0xffffffffu, incl, off);
    if (lane + off < 32) incl += x;
  }
  const int above = incl - s;
  const bool hit = above < rem && rem <= incl;
  int b = 0, r = 0, e = 0, cc = above;
  bool done = false;
#pragma unroll
  for (int j = 7; j >= 0; --j) {
    if (!done && cc + c[j] >= rem) {
      b = lane * 8 + j;
      r = rem - cc;
      e = c[j];
      done = true;
    }
    cc += c[j];
  }
  const uint32_t bal = __ballot_sync(0xffffffffu, hit);
  const int src = bal ? __ffs(bal) - 1 : 0;
  *bin = __shfl_sync(0xffffffffu, b, src);
  *rem_out = __shfl_sync(0xffffffffu, r, src);
  *eq_out = __shfl_sync(0xffffffffu, e, src);
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

// ---- block-wide merge sort, descending, of P (a power of two >= 64) DISTINCT 64-bit entries.
// Warps sort 64-entry runs in registers; then runs are merged pairwise, log2(P / 64) times: every
// entry finds by binary search how many entries of the sibling run precede it, which with its
// own index in its run is its place in the merged run.  One barrier per level (a bitonic
// network needs one per stride).  Reads buf, ping-pongs with alt, leaves the result in buf.
__device__ __forceinline__ void block_merge_sort_desc(unsigned long long* buf, unsigned long long* alt, int P) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int nwarps = blockDim.x >> 5;
  int levels = 0;
  while ((64 << levels) < P) ++levels;
  unsigned long long* src = (levels & 1) ? alt : buf;     // an even number of moves ends in buf
  unsigned long long* dst = (levels & 1) ? buf : alt;
  for (int blk = warp; blk < (P >> 6); blk += nwarps) {
    const int pos_a = blk * 64 + lane;
    unsigned long long a = buf[pos_a], b = buf[pos_a + 32];
    for (int size = 2; size <= 64; size <<= 1) warp_sort_steps(a, b, lane, size, size >> 1);   // every run descending
    src[pos_a] = a;
    src[pos_a + 32] = b;
  }
  __syncthreads();
  for (int lg = 6; (1 << lg) < P; ++lg) {
    const int L = 1 << lg;
#pragma unroll 2
    for (int i = tid; i < P; i += blockDim.x) {
      const unsigned long long e = src[i];
      const int run = i >> lg, within = i & (L - 1);
      const unsigned long long* sib = src + (run ^ 1) * L;
      int cnt = 0;                                   // sibling entries greater than e
      for (int step = L >> 1; step > 0; step >>= 1)
        if (sib[cnt + step - 1] > e) cnt += step;
      if (sib[cnt] > e) ++cnt;
      // equal entries do not occur; between the two runs of a pair the left one would go first
      dst[(run & ~1) * L + within + cnt] = e;
    }
    __syncthreads();
    unsigned long long* t = src; src = dst; dst = t;
  }
}

__global__ void __launch_bounds__(2 * kSelMaxThreads, 1) select_kernel(SelectParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  uint32_t* hist = reinterpret_cast<uint32_t*>(smem_raw);                     // kHistWords
  uint32_t* misc = hist + kHistWords;                                         // kSelMiscWords
  unsigned long long* cand = reinterpret_cast<unsigned long long*>(misc + kSelMiscWords);  // cand_cap
  uint32_t* bm = reinterpret_cast<uint32_t*>(cand + p.cand_cap);              // position bitmaps behind the list
  uint32_t* ws = misc + 8;                                                    // scan scratch (68 words)

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nt = blockDim.x;
  const int unit = blockIdx.x * p.unit_mul;
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
  // 16-byte groups: g[a0 + 4 i .. a0 + 4 i + 3], i < nb4; the few logits before and after are
  // handled one by one
  const int a0 = min(n, (4 - (int)(((long long)unit * p.ld + lo) & 3)) & 3);
  const int nb4 = (n - a0) >> 2;
  const float4* g4 = reinterpret_cast<const float4*>(g + a0);

  // full-softmax log-sum-exp from the scoring pass' per-chunk partials (of every head of the group)
  for (int j = warp; j < p.unit_mul; j += (nt >> 5)) {
    float mm = -INFINITY, ll = 0.f;
    const int nch = p.chunk_rows > 0 ? min(p.nchunks, (t + p.chunk_rows - 1) / p.chunk_rows) : p.nchunks;
    for (int c = lane; c < nch; c += 32) {
      const float2 x = p.part_ml[(long long)(unit + j) * p.nchunks + c];
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
      p.lse_full[unit + j] = lse;
      if (p.out_lse_full) p.out_lse_full[unit + j] = lse;
    }
  }
  if (tid == 0) {
    if ((unit % p.num_q_heads) == 0) p.anchor_t[b] = t;
    misc[4] = 0u;   // winners kept
    misc[5] = 0u;   // candidates listed
  }
  __syncthreads();

  int total = 0;          // entries in cand to sort; the first kk after sorting are S*
  bool fast_ok = false;
  if (kk > 0) {
    // ---------------- fast path
    // the histograms of the four 8-bit passes of step 3 (the barrier after step 2 covers this)
    for (int i = tid; i < kHistWords; i += nt) hist[i] = 0u;
    // 1. conservative threshold from a sample (or -inf: list everything).  Every warp takes a
    //    stratified 1-in-16 sample of 32-byte sectors spread over the whole range
    //    and finds, by bisection on the top 13 key bits, the value that
    //    1.75 k/16 + 16 sampled logits of the CTA would reach if all warps saw the same
    //    distribution; the lower median of the warps' values is the threshold.
    float thr = -INFINITY;
    // sample whenever listing every candidate would be much more than the ~2 k the threshold lets
    // through (always when they would not fit)
    if (n > p.cand_cap || (n >= 2048 && n > 4 * kk)) {
      const int nw = nt >> 5;
      // whole 32-byte sectors, one out of every sec_stride (>= 16: a 1-in-16 sample), at most two
      // per thread
      const int a8 = (8 - (int)(((long long)unit * p.ld + lo) & 7)) & 7;
      const int nsec = (n - a8) >> 3;
      const int sec_stride = max(kSampleStride, (nsec + 2 * nt - 1) / (2 * nt));
      const int S = nsec / sec_stride;               // sampled sectors
      const int slot = lane * nw + warp;
      // sampled logits that should reach the threshold: 1.75 x the expected number above the
      // k-th logit, plus 16; but no more than would fill 85 % of the list (a long context with a
      // large budget leaves little room: better a thinner margin than a certain overflow)
      int want = (int)((7ll * kk * 8 * S) / (4ll * n)) + 16;
      const int room = (int)((17ll * p.cand_cap * 8 * S) / (20ll * n));
      const bool tight = want > room;
      if (tight) want = max(room, (int)((8ll * kk * S) / n) + 1);
      const int rw = tight ? max(1, want / nw) : (want + nw - 1) / nw;   // per warp; rounded towards the room
      uint32_t prefix;
      if (2 * S <= nt) prefix = sample_quantile_half(g + a8, S, sec_stride, nw, rw);
      else if (S <= nt) prefix = sample_quantile<1>(g + a8, S, sec_stride, nt, slot, rw);
      else prefix = sample_quantile<2>(g + a8, S, sec_stride, nt, slot, rw);
      if (lane == 0) misc[80 + warp] = prefix;
      __syncthreads();
      const uint32_t mine = lane < nw ? misc[80 + lane] : 0xffffffffu;
      int rank = 0;
      for (int j = 0; j < nw; ++j) {
        const uint32_t o = __shfl_sync(0xffffffffu, mine, j);
        rank += (o < mine || (o == mine && j < lane)) ? 1 : 0;
      }
      const uint32_t pick = __ballot_sync(0xffffffffu, lane < nw && rank == (nw - 1) / 2);
      thr = key_to_float(__shfl_sync(0xffffffffu, mine, __ffs(pick) - 1));
      if (!(thr == thr)) thr = -INFINITY;
    }
    // 2. one pass over the logits: four 16-byte loads in flight per thread, a float compare per
    //    logit, then one warp scan and one shared-memory atomic per warp and batch to place the
    //    positions of the listed logits (their keys are fetched afterwards)
    if (warp == 0) {     // the logits before the first and after the last 16-byte group
      const int tail0 = a0 + 4 * nb4;
      int i = -1;
      if (lane < a0) i = lane;
      else if (lane >= 4 && tail0 + (lane - 4) < n) i = tail0 + (lane - 4);
      float v = -INFINITY;
      if (i >= 0) v = __ldcg(g + i);
      warp_append(i >= 0 && v >= thr, (unsigned long long)(uint32_t)(lo + i), cand, &misc[5],
                  (uint32_t)p.cand_cap);
    }
    for (int i0 = 0; i0 < nb4; i0 += 4 * nt) {
      float4 v[4];
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        const int i4 = i0 + x * nt + tid;
        v[x] = i4 < nb4 ? __ldcg(g4 + i4) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      }
      uint32_t cmask = 0u;
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        cmask |= (uint32_t)(v[x].x >= thr) << (4 * x);
        cmask |= (uint32_t)(v[x].y >= thr) << (4 * x + 1);
        cmask |= (uint32_t)(v[x].z >= thr) << (4 * x + 2);
        cmask |= (uint32_t)(v[x].w >= thr) << (4 * x + 3);
      }
      if (i0 + 4 * nt > nb4) {          // last batch: drop the groups past the end
#pragma unroll
        for (int x = 0; x < 4; ++x)
          if (i0 + x * nt + tid >= nb4) cmask &= ~(0xfu << (4 * x));
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
      const int pos0 = lo + a0 + 4 * (i0 + tid);
      while (cmask) {
        const int x = __ffs(cmask) - 1;
        cmask &= cmask - 1u;
        if (oc < (uint32_t)p.cand_cap)
          cand[oc] = (unsigned long long)(uint32_t)(pos0 + 4 * (x >> 2) * nt + (x & 3));
        ++oc;
      }
    }
    __syncthreads();
    const int ncand = (int)misc[5];
    fast_ok = ncand >= kk && ncand <= p.cand_cap;
    if (fast_ok) {
      // 3. exact radix select on the list: four 8-bit passes, one barrier each; every warp finds
      //    the digit for itself.  The first pass also fetches the keys of the listed positions.
      const float* srow = p.scores + (long long)unit * p.ld;
      for (int i0 = 0; i0 < ncand; i0 += nt) {
        const int i = i0 + tid;
        uint32_t key = 0u;
        if (i < ncand) {
          const int pos = (int)(uint32_t)cand[i];
          key = float_to_key(__ldcg(srow + pos));
          cand[i] = make_entry(key, pos);
        }
        hist_add(hist, key >> 24, i < ncand);
      }
      __syncthreads();
      uint32_t T = 0u;
      int rem = kk, eq = 0;
      for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t* h = hist + 256 * pass;
        if (pass > 0) {
          const uint32_t mask = 0xffffffffu << (shift + 8);
          for (int i0 = 0; i0 < ncand; i0 += nt) {
            const int i = i0 + tid;
            const uint32_t key = i < ncand ? (uint32_t)(cand[i] >> 32) : 0u;
            hist_add(hist + 256 * pass, (key >> shift) & 255u, i < ncand && (key & mask) == T);
          }
          __syncthreads();
        }
        int bin;
        find_bin_warp256(h, rem, &bin, &rem, &eq);
        T |= (uint32_t)bin << shift;
        if (rem == eq) break;      // every key that starts like T is needed: the low bits stay zero
      }
      // 4. winners and ties (keys >= T) to the front of the list, in place: a batch of entries
      //    is read by all threads before any of them is overwritten, and later batches lie
      //    behind everything written.  Sorting orders ties by position; the surplus ties fall
      //    behind the first kk entries.
      for (int c0 = 0; c0 < ncand; c0 += 8 * nt) {
        unsigned long long e[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const int i = c0 + x * nt + tid;
          e[x] = i < ncand ? cand[i] : 0ull;
        }
        __syncthreads();
#pragma unroll
        for (int x = 0; x < 8; ++x)
          if (c0 + x * nt < ncand)
            warp_append(e[x] != 0ull && (uint32_t)(e[x] >> 32) >= T, e[x], cand, &misc[4], (uint32_t)p.sort_cap);
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
        for (int i0 = 0; i0 < n; i0 += nt) {
          const int i = i0 + tid;
          const uint32_t u = i < n ? float_to_key(__ldcg(g + i)) : 0u;
          hist_add(hist, (u >> shift) & 255u, i < n && (u & mask) == prefix);
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
      for (int i0 = 0; i0 < n; i0 += nt) {
        const int i = i0 + tid;
        uint32_t u = 0u;
        if (i < n) u = float_to_key(__ldcg(g + i));
        warp_append(i < n && (u > T || (all_ties && u == T)), make_entry(u, lo + i), cand, &misc[4],
                    (uint32_t)p.sort_cap);
      }
      if (!all_ties) {
        // ties at T, lowest positions first
        int base = 0;
        for (int c0 = 0; c0 < n && base < need; c0 += nt) {
          const int i = c0 + tid;
          const bool f = (i < n) && float_to_key(__ldcg(g + i)) == T;
          const uint32_t bal = __ballot_sync(0xffffffffu, f);
          if (lane == 0) misc[8 + warp] = __popc(bal);
          __syncthreads();
          int before = 0, tot = 0;
          for (int w = 0; w < (nt >> 5); ++w) {
            const int c = (int)misc[8 + w];
            if (w < warp) before += c;
            tot += c;
          }
          const int rank = base + before + __popc(bal & ((1u << lane) - 1u));
          if (f && rank < need) cand[gt_total + rank] = make_entry(T, lo + i);
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
  for (int i = total + tid; i < P; i += nt) cand[i] = (unsigned long long)(P - i);   // distinct, below every entry
  const int words = (t + 31) >> 5;
  const int bm_words = p.two_bitmaps ? 2 * words : words;
  for (int w = tid; w < bm_words; w += nt) bm[w] = 0u;
  __syncthreads();
  if (p.sort_cap + P <= p.cand_cap) block_merge_sort_desc(cand, cand + p.sort_cap, P);
  else block_sort_desc(cand, P);

  // ---- S* in descending-logit order
  int* sd = p.sstar_desc + sunit * p.max_k;
  for (int e = tid; e < p.max_k; e += nt) {
    const int v = e < kk ? (int)(0xffffffffu - (uint32_t)(cand[e] & 0xffffffffull)) : -1;
    sd[e] = v;
    if (p.out_idx)
      for (int j = 0; j < p.unit_mul; ++j) p.out_idx[(long long)(unit + j) * p.max_k + e] = v;
  }
  if (tid == 0) {
    p.n_star[sunit] = kk;
    if (p.out_count)
      for (int j = 0; j < p.unit_mul; ++j) p.out_count[unit + j] = kk;
  }

  // ---- ascending S*, and the dilated S^ (Eq. 10), through position bitmaps
  if (p.two_bitmaps) {
    uint32_t* bh = bm + words;
    for (int e = tid; e < kk; e += nt) {
      const int pos = (int)(0xffffffffu - (uint32_t)(cand[e] & 0xffffffffull));
      atomicOr(&bm[pos >> 5], 1u << (pos & 31));
      const int rr = e < m_eff ? p.r : 0;
      for (int j = -rr; j <= rr; ++j) {
        const int x = pos + j;
        if (x >= 0 && x < t) atomicOr(&bh[x >> 5], 1u << (x & 31));
      }
    }
    __syncthreads();
    int ns, nh;
    compact_two(bm, bh, words, p.sstar_asc + sunit * p.max_k, p.max_k, p.shat_asc + sunit * p.shat_cap,
                p.shat_cap, ws, &ns, &nh);
    if (tid == 0) p.n_hat[sunit] = min(nh, p.shat_cap);
    return;
  }
  for (int e = tid; e < kk; e += nt) {
    const uint32_t pos = 0xffffffffu - (uint32_t)(cand[e] & 0xffffffffull);
    atomicOr(&bm[pos >> 5], 1u << (pos & 31u));
  }
  __syncthreads();
  compact_bitmap(bm, words, p.sstar_asc + sunit * p.max_k, p.max_k, ws);
  __syncthreads();   // every thread has finished reading the bitmap before it grows
  for (int e = tid; e < m_eff; e += nt) {
    const int pos = (int)(0xffffffffu - (uint32_t)(cand[e] & 0xffffffffull));
    for (int j = -p.r; j <= p.r; ++j) {
      const int x = pos + j;
      if (x >= 0 && x < t) atomicOr(&bm[x >> 5], 1u << (x & 31));
    }
  }
  __syncthreads();
  const int nh = compact_bitmap(bm, words, p.shat_asc + sunit * p.shat_cap, p.shat_cap, ws);
  if (tid == 0) p.n_hat[sunit] = min(nh, p.shat_cap);
}

}  // namespace prhs
