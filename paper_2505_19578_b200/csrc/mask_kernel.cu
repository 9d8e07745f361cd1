// Importance map -> block mask and compacted key-block lists.
//
// Algorithm "Construct Pivotal Pattern": sort the scores, find the smallest
// budget K whose top-K sum reaches gamma, select those indices.  Applied to each
// row-block independently over its causal entries.
//
// One warp owns one row.  The row's (score, index) pairs are packed into 64-bit
// keys, sorted with a bitonic network held entirely in registers (in-lane
// compare-exchanges for short distances, shuffles for long ones), scanned in
// float64, cut at gamma, and the selected indices are compacted in ascending
// order through a shared-memory bitmap + popcount prefix.
#include "common.cuh"

namespace sp {
namespace {

constexpr int kWarpsPerBlock = 4;
constexpr int kBitmapWords = kMaxNb / 32;

// Sort key: ascending order of the key == descending score, then ascending index.
// Scores are finite and >= 0, so their bit patterns order like the values.
__device__ __forceinline__ uint64_t make_key(float v, int idx) {
  uint32_t bits = (v > 0.f && v <= 3.4028235e38f) ? __float_as_uint(v) : 0u;
  return ((uint64_t)(~bits) << 32) | (uint32_t)idx;
}
__device__ __forceinline__ float key_score(uint64_t key) { return __uint_as_float(~(uint32_t)(key >> 32)); }

__device__ __forceinline__ uint64_t shfl_xor_u64(uint64_t x, int m) {
  uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)x, m);
  uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(x >> 32), m);
  return ((uint64_t)hi << 32) | lo;
}

// Bitonic sort of 32*E keys spread over a warp; sorted position p lives in
// lane p / E, register p % E.
template <int E>
__device__ __forceinline__ void warp_bitonic_sort(uint64_t (&key)[E], int lane) {
#pragma unroll
  for (int k = 2; k <= 32 * E; k <<= 1) {
#pragma unroll
    for (int d = k >> 1; d > 0; d >>= 1) {
      if (d < E) {
#pragma unroll
        for (int e = 0; e < E; ++e) {
          if ((e & d) == 0) {
            const int p = lane * E + e;
            const bool up = (p & k) == 0;
            uint64_t a = key[e], b = key[e | d];
            const bool sw = (a > b) == up;
            key[e] = sw ? b : a;
            key[e | d] = sw ? a : b;
          }
        }
      } else {
        const int lm = d / E;
        const bool lower = (lane & lm) == 0;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const int p = lane * E + e;
          const bool up = (p & k) == 0;
          uint64_t other = shfl_xor_u64(key[e], lm);
          uint64_t mn = key[e] < other ? key[e] : other;
          uint64_t mx = key[e] < other ? other : key[e];
          key[e] = (lower == up) ? mn : mx;
        }
      }
    }
  }
}

template <int E>
__device__ void mask_row(const float* __restrict__ row, int n, int nb, double gamma, uint8_t* mask_row_out,
                         int32_t* count_out, int32_t* idx_row_out, uint32_t* bitmap, int lane) {
  uint64_t key[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int j = e * 32 + lane;             // coalesced load; the sort does not care where a key starts
    key[e] = j < n ? make_key(row[j], j) : ~0ull;
  }
  warp_bitonic_sort<E>(key, lane);

  // running sum in sorted order, float64
  double val[E];
  double local = 0.0;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    val[e] = key[e] != ~0ull ? (double)key_score(key[e]) : 0.0;
    local += val[e];
  }
  double incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  double cum = incl - local;
  int first = -1;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    cum += val[e];
    if (first < 0 && key[e] != ~0ull && cum >= gamma) first = lane * E + e;
  }
  const unsigned hit = __ballot_sync(0xffffffffu, first >= 0);
  int K = n;
  if (hit) K = __shfl_sync(0xffffffffu, first, __ffs(hit) - 1) + 1;

  // selected set -> bitmap over key-block indices
  if (lane < kBitmapWords) bitmap[lane] = 0u;
  __syncwarp();
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int p = lane * E + e;
    if (p < K) {
      const uint32_t j = (uint32_t)key[e];
      atomicOr(&bitmap[j >> 5], 1u << (j & 31));
    }
  }
  __syncwarp();

  // ascending compaction
  uint32_t word = lane < kBitmapWords ? bitmap[lane] : 0u;
  int c = __popc(word), off = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int t = __shfl_up_sync(0xffffffffu, off, o);
    if (lane >= o) off += t;
  }
  off -= c;
  while (word) {
    const int b = __ffs(word) - 1;
    idx_row_out[off++] = lane * 32 + b;
    word &= word - 1;
  }
  for (int j = K + lane; j < nb; j += 32) idx_row_out[j] = -1;
  if (lane == 0) *count_out = K;
  if (mask_row_out)
    for (int j = lane; j < nb; j += 32) mask_row_out[j] = (uint8_t)((bitmap[j >> 5] >> (j & 31)) & 1u);
  __syncwarp();
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32) block_mask_kernel(const MaskArgs a) {
  __shared__ uint32_t bitmaps[kWarpsPerBlock][kBitmapWords];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long total = (long)a.n_maps * a.nb;
  for (long w = (long)blockIdx.x * kWarpsPerBlock + warp; w < total; w += (long)gridDim.x * kWarpsPerBlock) {
    const int i = a.nb - 1 - (int)(w / a.n_maps);   // long rows first
    const int mp = (int)(w % a.n_maps);
    const size_t rbase = ((size_t)mp * a.nb + i) * a.nb;
    const float* row = a.importance + rbase;
    uint8_t* mrow = a.mask ? a.mask + rbase : nullptr;
    int32_t* cnt = a.counts + (size_t)mp * a.nb + i;
    int32_t* irow = a.indices + rbase;
    const int n = i + 1;
    uint32_t* bm = bitmaps[warp];
    if (n <= 32)        mask_row<1>(row, n, a.nb, a.gamma, mrow, cnt, irow, bm, lane);
    else if (n <= 64)   mask_row<2>(row, n, a.nb, a.gamma, mrow, cnt, irow, bm, lane);
    else if (n <= 128)  mask_row<4>(row, n, a.nb, a.gamma, mrow, cnt, irow, bm, lane);
    else if (n <= 256)  mask_row<8>(row, n, a.nb, a.gamma, mrow, cnt, irow, bm, lane);
    else if (n <= 512)  mask_row<16>(row, n, a.nb, a.gamma, mrow, cnt, irow, bm, lane);
    else                mask_row<32>(row, n, a.nb, a.gamma, mrow, cnt, irow, bm, lane);
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
