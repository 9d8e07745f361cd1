// Importance map -> block mask and compacted key-block lists.
//
// Algorithm "Construct Pivotal Pattern": sort the scores, find the smallest
// budget K whose top-K sum reaches gamma, select those indices.  Applied to each
// row-block independently over its causal entries.
//
// One warp owns one row, its scores in registers (lane l holds entries l, l + 32,
// ...).  No sort is needed to know WHICH entries the sorted prefix holds: with
// T the largest score for which the entries >= T sum to at least gamma, the
// prefix is every entry above T plus the first few entries equal to T in index
// order (equal scores go to the smaller key-block).  T is found bit by bit on
// the fp32 bit patterns (31 passes of a compare, an add and a warp reduction per
// held entry); the sums are exact fixed-point integers in units of 2^-50 (scores
// are probabilities: every score >= 2^-27 is represented exactly, smaller ones
// lose less than 2^-50 each; a score above 4 counts as 4), and integer additions
// commute, so the result does not depend on the order of the additions.  The
// selected entries are then written in ascending index order with ballots.
// A full sort of (score, index) keys in registers (a bitonic network of 55
// stages for 1024 keys) did the same in three times the instructions.
#include "common.cuh"

namespace sp {
namespace {

constexpr int kWarpsPerBlock = 4;
constexpr unsigned long long kFxCap = 1ull << 52;   // 4.0 in units of 2^-50: 1024 of them still fit in 64 bits

// Finite positive scores only; anything else counts as 0.
__device__ __forceinline__ uint32_t mask_score_bits(float v) { return (v > 0.f && v <= 3.4028235e38f) ? __float_as_uint(v) : 0u; }

// value * 2^50 of a positive finite fp32 bit pattern (bits below 2^-50 dropped, capped at kFxCap): integer shifts only
__device__ __forceinline__ unsigned long long mask_score_fixed(uint32_t bits) {
  const int e = (int)(bits >> 23);
  const unsigned long long m = (unsigned long long)(bits & 0x7FFFFFu) | (e ? 0x800000ull : 0ull);
  const int sh = (e ? e : 1) - 150 + 50;          // value = m * 2^((e ? e : 1) - 150)
  if (sh >= 29) return kFxCap;                    // m < 2^24, so m << 29 could pass the cap
  if (sh >= 0) { const unsigned long long x = m << sh; return x < kFxCap ? x : kFxCap; }
  return sh > -64 ? m >> (-sh) : 0ull;
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int E>
__device__ void mask_row(const float* __restrict__ row, int n, int nb, unsigned long long gamma_fx, uint8_t* mask_row_out,
                         int32_t* count_out, int32_t* idx_row_out, int lane) {
  uint32_t bits[E];
  unsigned long long fx[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int j = e * 32 + lane;
    bits[e] = j < n ? mask_score_bits(row[j]) : 0u;
    fx[e] = mask_score_fixed(bits[e]);
  }
  auto sum_from = [&](uint32_t t) {
    unsigned long long s = 0;
#pragma unroll
    for (int e = 0; e < E; ++e)
      if (bits[e] >= t) s += fx[e];
    return warp_sum_u64(s);
  };
  const unsigned long long total = sum_from(1u);
  const bool all = total < gamma_fx;              // the scores never reach gamma: every causal entry is selected
  uint32_t T = 0u, k_eq = 0u;
  if (!all) {
#pragma unroll 1
    for (int bit = 30; bit >= 0; --bit) {
      const uint32_t cand = T | (1u << bit);
      if (sum_from(cand) >= gamma_fx) T = cand;
    }
    const unsigned long long above = sum_from(T + 1u);
    const unsigned long long v_fx = mask_score_fixed(T);
    const unsigned long long need = gamma_fx > above ? gamma_fx - above : 1ull;
    const unsigned long long k = v_fx ? (need + v_fx - 1) / v_fx : ~0ull;
    k_eq = k > 0xffffffffull ? 0xffffffffu : (uint32_t)k;
  }
  // selection in ascending index order: everything above T, then copies of T while they are needed
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t seen_eq = 0u;
  int cnt = 0;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int j = e * 32 + lane;
    const bool eq = !all && bits[e] == T && j < n;
    const uint32_t bal_eq = __ballot_sync(0xffffffffu, eq);
    const bool on = j < n && (all || bits[e] > T || (eq && seen_eq + __popc(bal_eq & lt) < k_eq));
    seen_eq += __popc(bal_eq);
    const uint32_t bal = __ballot_sync(0xffffffffu, on);
    if (on) idx_row_out[cnt + __popc(bal & lt)] = j;
    cnt += __popc(bal);
    if (mask_row_out && j < nb) mask_row_out[j] = (uint8_t)(on ? 1 : 0);
  }
  for (int j = cnt + lane; j < nb; j += 32) idx_row_out[j] = -1;
  if (mask_row_out)
    for (int j = E * 32 + lane; j < nb; j += 32) mask_row_out[j] = 0;
  if (lane == 0) *count_out = cnt;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32) block_mask_kernel(const MaskArgs a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long total = (long)a.n_maps * a.nb;
  // cumulative >= gamma  <=>  fixed-point cumulative >= ceil(gamma * 2^50)
  const double gs = a.gamma * 1125899906842624.0;
  const unsigned long long gamma_fx = gs >= 9.0e18 ? ~0ull : (gs <= 1.0 ? 1ull : (unsigned long long)ceil(gs));
  for (long w = (long)blockIdx.x * kWarpsPerBlock + warp; w < total; w += (long)gridDim.x * kWarpsPerBlock) {
    const int i = a.nb - 1 - (int)(w / a.n_maps);   // long rows first
    const int mp = (int)(w % a.n_maps);
    const size_t rbase = ((size_t)mp * a.nb + i) * a.nb;
    const float* row = a.importance + rbase;
    uint8_t* mrow = a.mask ? a.mask + rbase : nullptr;
    int32_t* cnt = a.counts + (size_t)mp * a.nb + i;
    int32_t* irow = a.indices + rbase;
    const int n = i + 1;
    if (n <= 32)        mask_row<1>(row, n, a.nb, gamma_fx, mrow, cnt, irow, lane);
    else if (n <= 64)   mask_row<2>(row, n, a.nb, gamma_fx, mrow, cnt, irow, lane);
    else if (n <= 128)  mask_row<4>(row, n, a.nb, gamma_fx, mrow, cnt, irow, lane);
    else if (n <= 256)  mask_row<8>(row, n, a.nb, gamma_fx, mrow, cnt, irow, lane);
    else if (n <= 512)  mask_row<16>(row, n, a.nb, gamma_fx, mrow, cnt, irow, lane);
    else                mask_row<32>(row, n, a.nb, gamma_fx, mrow, cnt, irow, lane);
  }
}

__global__ void fill_causal_mask_kernel(uint8_t* mask, int nb) {
  const int i = blockIdx.x;
  for (int j = threadIdx.x; j < nb; j += blockDim.x) mask[(size_t)i * nb + j] = j <= i ? 1 : 0;
}

}  // namespace

cudaError_t launch_block_mask(const MaskArgs& a, cudaStream_t s) {
  const long total = (long)a.n_maps * a.nb;
  if (total == 0) return cudaSuccess;
  const int blocks = (int)((total + kWarpsPerBlock - 1) / kWarpsPerBlock);
  block_mask_kernel<<<blocks, kWarpsPerBlock * 32, 0, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_fill_causal_mask(uint8_t* mask, int nb, cudaStream_t s) {
  fill_causal_mask_kernel<<<nb, 128, 0, s>>>(mask, nb);
  return cudaGetLastError();
}

}  // namespace sp
