// Shared device helpers for the PrHS sparse decode-attention kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace prhs {

constexpr int kHeadDim = 128;              // elements per K/V row
constexpr int kRowBytes = kHeadDim * 2;    // 256 B per bf16 row
constexpr int kPageShift = 4;              // 16 positions per page
constexpr float kScale = 0.08838834764831845f;        // 1 / sqrt(128)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

constexpr uint32_t kFlagBadIndex = 1u;
constexpr uint32_t kFlagBadPage = 2u;
constexpr uint32_t kFlagSelectFallback = 4u;

// Device-side copy of a KV view (see prhs_kv_view): element strides, optional page table.
struct KvDev {
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  long long stride_outer;
  long long stride_head;
  const int* page_table;
  int page_table_stride;
  const int* seq_lens;
  int num_pages;
};

// Which stored middle set a (b, h) unit attends over.  Sets live in slots: [unit][slot][stride]
// for S* (ascending) and for the dilated S^; a unit uses S* only on the step that retrieved
// it (and not even then with PRHS_DILATE_ANCHOR), else S^ (Def. 3.2).
struct SetRef {
  const int* star;        // S* ascending, [U][slots][star_stride]; nullptr = no fused set
  const int* n_star;      // [U][slots]
  const int* hat;         // S^ ascending, [U][slots][hat_stride]
  const int* n_hat;       // [U][slots]
  const int* slot_of;     // [U] slot each unit uses this step, or nullptr = slot 0
  const int* own_of;      // [U] != 0 where the unit retrieved this step, or nullptr = own_all
  int star_stride, hat_stride, slots, own_all;
  int share_gq;           // > 1: the heads of a KV group share the set stored for the group's first head
  int sinks, window;
  double psaw_c;          // sliding-window factor of this layer (0 = off)
};

// The unit's middle set M (ascending, unique) and its length.
__device__ __forceinline__ const int* middle_of(const SetRef& r, int unit, int* n, int* stride) {
  if (r.share_gq > 1) unit -= unit % r.share_gq;      // units are b * Hq + h and Hq is a multiple of the group
  const int slot = r.slot_of ? __ldg(r.slot_of + unit) : 0;
  const bool own = r.own_of ? (__ldg(r.own_of + unit) != 0) : (r.own_all != 0);
  const long long e = (long long)unit * r.slots + slot;
  if (own) {
    *n = min(__ldg(r.n_star + e), r.star_stride);
    *stride = r.star_stride;
    return r.star + e * r.star_stride;
  }
  *n = min(__ldg(r.n_hat + e), r.hat_stride);
  *stride = r.hat_stride;
  return r.hat + e * r.hat_stride;
}

// Start of the progressive sliding attention window (Eq. 11): P = floor(c * t) with
// c = 1 - phi^(alpha (l - l_s) / (N - l_s)) computed on the host in double (0 = no window).
__device__ __forceinline__ int psaw_start(double c, int t) {
  if (c <= 0.0) return 0;
  const int p = (int)floor(c * (double)t);
  return max(0, min(p, t));
}

// bf16 pair (packed in 32 bits) -> two floats; exact.
__device__ __forceinline__ float bf_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

// Order-preserving map fp32 -> uint32: larger float <=> larger key (-0 < +0, NaNs at the ends).
__device__ __forceinline__ uint32_t float_to_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Inverse of float_to_key.
__device__ __forceinline__ float key_to_float(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Combine two online-softmax states kept in the log2 domain: (m, l) <- (m, l) (+) (m2, l2).
__device__ __forceinline__ void ml_combine(float& m, float& l, float m2, float l2) {
  float mn = fmaxf(m, m2);
  if (mn == -INFINITY) return;
  l = l * exp2f(m - mn) + l2 * exp2f(m2 - mn);
  m = mn;
}

}  // namespace prhs
