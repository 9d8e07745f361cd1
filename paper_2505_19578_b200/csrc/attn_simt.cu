// Plain fp32 CUDA-core attention kernel: one warp per query row, no tensor
// cores, no shared K/V staging.  It exists as an independent on-device
// cross-check of the tensor-core kernel (different algorithm for the block
// importance: two passes with the final log-sum-exp instead of one pass with
// spilled statistics).  It is not the product path.
//
// Computes, for every listed head and row-block i, softmax over the selected
// key-blocks (causal inside the diagonal block) times V  (Section 5.1, masked
// attention), and optionally the tile masses of the block-importance map.
#include <math_constants.h>

#include "common.cuh"

namespace sp {
namespace {

constexpr int kWarps = 4;

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

template <int D>
__device__ __forceinline__ float dot_row(const float* qs, const __nv_bfloat16* krow) {
  const uint4* kv = reinterpret_cast<const uint4*>(krow);
  float acc = 0.f;
#pragma unroll
  for (int x = 0; x < D / 8; ++x) {
    uint4 u = __ldg(kv + x);
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      float2 f = __bfloat1622float2(h2[y]);
      acc = fmaf(qs[x * 8 + 2 * y], f.x, acc);
      acc = fmaf(qs[x * 8 + 2 * y + 1], f.y, acc);
    }
  }
  return acc;
}

template <int D>
__global__ void __launch_bounds__(kWarps * 32) attn_simt_kernel(const AttnArgs a) {
  extern __shared__ float smem[];
  float* qs_all = smem;                       // [kWarps][D]
  float* macc = smem + kWarps * D;            // [kWarps][Nb] tile-mass partials (importance only)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = a.Nb - 1 - (int)blockIdx.x;   // heavy row-blocks first
  const int slot = blockIdx.y;
  const int h = a.heads.v[slot];
  const int g = h / a.group;
  const int list = a.lists_dev ? a.lists_dev[slot] : a.lists.v[slot];   // decided on the device, or by the host
  const int B = a.B;
  const int cnt = list >= 0 ? a.counts[(size_t)list * a.Nb + i] : i + 1;
  const int32_t* idx = list >= 0 ? a.indices + ((size_t)list * a.Nb + i) * a.Nb : nullptr;
  const __nv_bfloat16* Kg = a.k + (size_t)g * a.k_sh;
  const __nv_bfloat16* Vg = a.v + (size_t)g * a.v_sh;
  float* qs = qs_all + warp * D;
  const bool want_imp = a.importance != nullptr;

  if (want_imp)
    for (int j = lane; j < a.Nb; j += 32) macc[warp * a.Nb + j] = 0.f;
  __syncwarp();

  for (int row = warp; row < B; row += kWarps) {
    const int r = i * B + row;
    const __nv_bfloat16* qrow = a.q + (size_t)h * a.q_sh + (size_t)r * a.q_sn;
    for (int e = lane; e < D; e += 32) qs[e] = __bfloat162float(qrow[e]) * a.scale_log2;
    __syncwarp();

    float m = -CUDART_INF_F, l = 0.f;
    float o[D / 32];
#pragma unroll
    for (int e = 0; e < D / 32; ++e) o[e] = 0.f;

    for (int t = 0; t < cnt; ++t) {
      const int j = idx ? idx[t] : t;
      for (int c0 = j * B; c0 < (j + 1) * B && c0 <= r; c0 += 32) {
        const int c = c0 + lane;
        float s = -CUDART_INF_F;
        if (c <= r) s = dot_row<D>(qs, Kg + (size_t)c * a.k_sn);
        const float m_new = fmaxf(m, warp_max(s));      // lane c0 <= r is always finite
        const float p = exp2f(s - m_new);
        const float corr = exp2f(m - m_new);
        l = l * corr + warp_sum(p);
#pragma unroll
        for (int e = 0; e < D / 32; ++e) o[e] *= corr;
        for (int kk = 0; kk < 32; ++kk) {
          const float pk = __shfl_sync(0xffffffffu, p, kk);
          if (pk != 0.f) {
            const __nv_bfloat16* vrow = Vg + (size_t)(c0 + kk) * a.v_sn;
#pragma unroll
            for (int e = 0; e < D / 32; ++e) o[e] = fmaf(pk, __bfloat162float(vrow[lane + 32 * e]), o[e]);
          }
        }
        m = m_new;
      }
    }
    const float inv_l = 1.f / l;
    __nv_bfloat16* orow = a.o + (size_t)h * a.o_sh + (size_t)r * a.o_sn;
#pragma unroll
    for (int e = 0; e < D / 32; ++e) orow[lane + 32 * e] = __float2bfloat16_rn(o[e] * inv_l);
    const float lse2 = m + log2f(l);
    if (a.lse && lane == 0) a.lse[(size_t)slot * a.N + r] = lse2 * 0.6931471805599453f;

    if (want_imp) {
      // second pass: probabilities with the final log-sum-exp, summed per tile
      for (int t = 0; t < cnt; ++t) {
        const int j = idx ? idx[t] : t;
        float tile = 0.f;
        for (int c0 = j * B; c0 < (j + 1) * B && c0 <= r; c0 += 32) {
          const int c = c0 + lane;
          float p = 0.f;
          if (c <= r) p = exp2f(dot_row<D>(qs, Kg + (size_t)c * a.k_sn) - lse2);
          tile += p;
        }
        tile = warp_sum(tile);
        if (lane == 0) macc[warp * a.Nb + j] += tile;   // this warp's rows, in row order
      }
    }
    __syncwarp();
  }

  if (want_imp) {
    __syncthreads();
    float* out = a.importance + ((size_t)slot * a.Nb + i) * a.Nb;
    for (int j = threadIdx.x; j < a.Nb; j += blockDim.x) {
      float s = 0.f;
      if (j <= i)
        for (int w = 0; w < kWarps; ++w) s += macc[w * a.Nb + j];
      out[j] = s / (float)B;
    }
  }
}

}  // namespace

cudaError_t launch_attn_simt(const AttnArgs& a, cudaStream_t s) {
  dim3 grid(a.Nb, a.n_heads), block(kWarps * 32);
  size_t smem = (size_t)kWarps * a.d * sizeof(float) + (a.importance ? (size_t)kWarps * a.Nb * sizeof(float) : 0);
  if (a.d == 64)
    attn_simt_kernel<64><<<grid, block, smem, s>>>(a);
  else
    attn_simt_kernel<128><<<grid, block, smem, s>>>(a);
  return cudaGetLastError();
}

}  // namespace sp
