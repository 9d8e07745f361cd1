// Block-wide cumulative cut (the "minimum budget whose scores sum to gamma" of the paper's
// Algorithms "Construct Pivotal Pattern" and "Search Vertical Slash Pattern") without a sort.
//
// The scores are non-negative fp32 values; their bit patterns order like the values.  The cut value
// is the largest bit pattern T for which the normalised scores >= T sum to at least gamma; it is
// found bit by bit (31 passes over the data, each a block reduction).  Sums are taken in fixed
// point (the scores themselves, exactly, times 2^50; gamma is applied to their exact total): integer
// additions commute, so the result does not depend on which thread owns which score.
// The caller then marks every score above T and the first k_eq scores equal to T in its index order.
#pragma once

#include <stdint.h>

namespace sp {

struct CutResult {
  unsigned int cut_bits;   // bit pattern of the cut value
  unsigned int k_eq;       // how many scores equal to the cut value are selected (in index order)
  bool all;                // the scores never reach gamma: everything is selected
};

// value * 2^50 of a positive finite fp32 bit pattern, exactly (bits below 2^-50 are dropped): integer
// shifts only.  The callers' scores are softmax rows or sums of at most a block of probabilities, so a
// score is at most 2^7 and all of them together at most 2^13: every sum fits in 64 bits.
__device__ __forceinline__ unsigned long long score_fixed(unsigned int bits) {
  const int e = (int)(bits >> 23);
  const unsigned long long m = (unsigned long long)(bits & 0x7FFFFFu) | (e ? 0x800000ull : 0ull);
  const int sh = (e ? e : 1) - 150 + 50;          // value = m * 2^((e ? e : 1) - 150)
  if (sh >= 0) return sh < 38 ? m << sh : (m << 38);
  return sh > -64 ? m >> (-sh) : 0ull;
}

// Finite positive scores only; anything else counts as 0.
__device__ __forceinline__ unsigned int score_bits(float v) { return (v > 0.f && v <= 3.4028235e38f) ? __float_as_uint(v) : 0u; }

// Sum over the block (and, with REDUCE, over whatever wider group the caller's functor spans).
template <int THREADS>
__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* sh /*[THREADS/32 + 1]*/) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int w = 0; w < THREADS / 32; ++w) t += sh[w];
    sh[THREADS / 32] = t;
  }
  __syncthreads();
  return sh[THREADS / 32];
}

// for_each(f): calls f(float score) for every score this thread owns (the same scores on every call).
// widen(x): turns this block's sum into the sum over all blocks that share the vector (identity for one block).
template <int THREADS, class ForEach, class Widen>
__device__ CutResult block_cumulative_cut(ForEach for_each, Widen widen, double gamma, unsigned long long* sh /*[THREADS/32 + 1]*/) {
  auto sum_from = [&](unsigned int t_bits) {
    unsigned long long s = 0;
    for_each([&](float v) {
      const unsigned int b = score_bits(v);
      if (b >= t_bits) s += score_fixed(b);
    });
    return widen(block_sum_u64<THREADS>(s, sh));
  };
  CutResult r{0u, 0u, false};
  const unsigned long long total = sum_from(1u);
  // cumulative / total >= gamma  <=>  cumulative >= gamma * total (rounded up to the next integer)
  const double gt = gamma * (double)total;
  const unsigned long long gamma_fx = gt >= 1.8e19 ? ~0ull : (unsigned long long)ceil(gt);
  if (total == 0ull || total < gamma_fx) { r.all = true; return r; }
  unsigned int T = 0u;
  for (int bit = 30; bit >= 0; --bit) {
    const unsigned int cand = T | (1u << bit);
    if (sum_from(cand) >= gamma_fx) T = cand;
  }
  const unsigned long long above = sum_from(T + 1u);
  const unsigned long long v_fx = score_fixed(T);
  const unsigned long long need = gamma_fx > above ? gamma_fx - above : 1ull;   // the scores above T alone fall short
  const unsigned long long k = v_fx ? (need + v_fx - 1) / v_fx : 1ull;
  r.cut_bits = T;
  r.k_eq = k > 0xffffffffull ? 0xffffffffu : (k ? (unsigned int)k : 1u);
  return r;
}

}  // namespace sp
