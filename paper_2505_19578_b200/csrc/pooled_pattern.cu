// Paper-literal pattern construction and decision.
//
//   Section 5.2, "Sparse Attention Computation": next to the output the kernel
//   yields the block-wise average of the QK values, A~.
//   Algorithm "Construct Pivotal Pattern": A~ = softmax(A~); a~ = its last row;
//   flatten and normalise; sort; minimum budget K whose scores sum to gamma;
//   index set -> mask.
//   Algorithm "Determine Sparse Pattern": a^ = softmax(pool(Q^ K^T)/sqrt(d)) for
//   the last block of queries, d_sparse = sqrt(JSD(a^ || u)), d_sim =
//   sqrt(JSD(a^ || a~)); shared pivot iff d_sparse < delta and d_sim < tau.
//
// The average of q_r . k_c over a full block is the product of the block means
// of Q and of K, so the map needs no pass over the tiles: block means of Q and K
// (one read of the two tensors), one small product per block, and the diagonal
// block (only its visible half is averaged) through a running key prefix sum.
// The global cut needs no sort: the cut value is found bit by bit on the score bit
// patterns with exact fixed-point sums (select.cuh), followed by an ordered pass that
// breaks ties towards the smaller flattened index.  All of it is HBM- and latency-sized
// work (a few MB per head).
#include <cooperative_groups.h>
#include <math_constants.h>

#include "common.cuh"
#include "select.cuh"

namespace sp {
namespace {

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// The block means, their products, the softmax over them and the divergences are carried in float64: the
// global cut compares a cumulative sum of a million scores with gamma, and fp32 means and logits (of order 1..30)
// would move that sum by 1e-5; with float64 up to the scores (rounded to fp32 once) it moves by under 1e-7.
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_max(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---- block means of Q and K, and the average of the diagonal block ------------------------
// grid (Nb, n_heads), d threads: thread = one head-dim column.
__global__ void block_means_kernel(const PooledArgs a) {
  __shared__ double red[4];
  const int i = blockIdx.x, slot = blockIdx.y, col = threadIdx.x;
  const int h = a.heads.v[slot], g = h / a.group;
  const __nv_bfloat16* q = a.q + (size_t)h * a.q_sh + (size_t)i * a.B * a.q_sn + col;
  const __nv_bfloat16* k = a.k + (size_t)g * a.k_sh + (size_t)i * a.B * a.k_sn + col;
  double qsum = 0.0, kcum = 0.0, acc = 0.0;
  for (int r = 0; r < a.B; ++r) {
    const double qv = (double)__bfloat162float(q[(size_t)r * a.q_sn]);
    kcum += (double)__bfloat162float(k[(size_t)r * a.k_sn]);
    qsum += qv;
    acc = fma(qv, kcum, acc);           // q_r . (k_0 + ... + k_r): the visible half of the diagonal block
  }
  const double inv = 1.0 / (double)a.B;
  a.qbar[((size_t)slot * a.Nb + i) * a.d + col] = qsum * inv;
  a.kbar[((size_t)slot * a.Nb + i) * a.d + col] = kcum * inv;
  acc = warp_sum(acc);
  if ((col & 31) == 0) red[col >> 5] = acc;
  __syncthreads();
  if (col == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    a.diag[(size_t)slot * a.Nb + i] = t * a.scale / (0.5 * (double)a.B * (double)(a.B + 1));
  }
}

// ---- A~[i][j] = qbar_i . kbar_j / sqrt(d)  (j < i), diagonal from above, -inf for j > i ------
// grid (Nb, n_heads), 128 threads: warp w takes key-blocks w, w+4, ...
__global__ void pooled_logits_kernel(const PooledArgs a) {
  const int i = blockIdx.x, slot = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const double* qb = a.qbar + ((size_t)slot * a.Nb + i) * a.d;
  double* out = a.pooled + ((size_t)slot * a.Nb + i) * a.Nb;
  const int per = a.d / 32;              // 2 or 4 consecutive columns per lane
  double qv[4];
  for (int e = 0; e < per; ++e) qv[e] = qb[lane * per + e];
  for (int j = warp; j < i; j += 4) {
    const double* kb = a.kbar + ((size_t)slot * a.Nb + j) * a.d;
    double acc = 0.0;
    for (int e = 0; e < per; ++e) acc = fma(qv[e], kb[lane * per + e], acc);
    acc = warp_sum(acc);
    if (lane == 0) out[j] = acc * a.scale;
  }
  if (threadIdx.x == 0) out[i] = a.diag[(size_t)slot * a.Nb + i];
  for (int j = i + 1 + (int)threadIdx.x; j < a.Nb; j += blockDim.x) out[j] = -CUDART_INF;
}

// ---- row-wise softmax of the block averages; one warp per row -------------------------------
__global__ void pooled_softmax_kernel(const double* __restrict__ pooled, int n_maps, int nb, float* __restrict__ scores,
                                      float* __restrict__ last_row) {
  const int lane = threadIdx.x & 31;
  const long w = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (w >= (long)n_maps * nb) return;
  const int mp = (int)(w / nb), i = (int)(w % nb);
  const double* row = pooled + ((size_t)mp * nb + i) * nb;
  float* out = scores + ((size_t)mp * nb + i) * nb;
  double m = -CUDART_INF;
  for (int j = lane; j <= i; j += 32) m = fmax(m, row[j]);
  m = warp_max(m);
  double s = 0.0;
  for (int j = lane; j <= i; j += 32) s += exp(row[j] - m);
  s = warp_sum(s);
  const double inv = 1.0 / s;
  for (int j = lane; j < nb; j += 32) {
    const float p = j <= i ? (float)(exp(row[j] - m) * inv) : 0.f;      // the one rounding to fp32
    out[j] = p;
    if (last_row && i == nb - 1) last_row[(size_t)mp * nb + j] = p;
  }
}

// ---- global cumulative cut over one map; a cluster of 8 CTAs of 1024 threads per map --------
// Rows are dealt round-robin to the cluster's 256 warps (balanced: long and short rows alternate), lanes
// run along a row's existing blocks j <= i.  Each pass of the cut is a block sum widened to the cluster
// through distributed shared memory (every CTA reads the eight partial sums and adds them in the same
// order, so all of them take the same decisions).
constexpr int kSelThreads = 1024;
constexpr int kSelCluster = 8;

__global__ void __cluster_dims__(kSelCluster, 1, 1) __launch_bounds__(kSelThreads)
global_select_kernel(const float* __restrict__ scores, int nb, double gamma, uint8_t* __restrict__ mask) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ unsigned long long sh_sum[kSelThreads / 32 + 1];
  __shared__ unsigned long long partial[2];          // this CTA's sum of the current pass (double-buffered)
  __shared__ unsigned int row_eq[kMaxNb];            // copies of the cut value per row (every CTA holds all rows)
  __shared__ unsigned int scan_tmp[kSelThreads / 32];
  const int mp = blockIdx.y, rank = (int)cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kWarps = kSelThreads / 32, kStride = kWarps * kSelCluster;
  const float* sc = scores + (size_t)mp * nb * nb;
  uint8_t* mk = mask + (size_t)mp * nb * nb;
  const int row0 = rank * kWarps + warp;

  auto for_each = [&](auto f) {
    for (int i = row0; i < nb; i += kStride)
      for (int j = lane; j <= i; j += 32) f(sc[(size_t)i * nb + j]);
  };
  int pass = 0;
  auto widen = [&](unsigned long long x) {
    const int buf = pass & 1;
    ++pass;
    if (tid == 0) partial[buf] = x;
    cluster.sync();
    unsigned long long t = 0;
    for (int r = 0; r < kSelCluster; ++r) t += *cluster.map_shared_rank(&partial[buf], r);
    return t;
  };
  const CutResult cut = block_cumulative_cut<kSelThreads>(for_each, widen, gamma, sh_sum);

  // copies of the cut value per row, published to every CTA of the cluster
  for (int i = tid; i < nb; i += kSelThreads) row_eq[i] = 0u;
  cluster.sync();
  if (!cut.all)
    for (int i = row0; i < nb; i += kStride) {
      unsigned int n_eq = 0;
      for (int j0 = 0; j0 <= i; j0 += 32) {
        const int j = j0 + lane;
        n_eq += __popc(__ballot_sync(0xffffffffu, j <= i && score_bits(sc[(size_t)i * nb + j]) == cut.cut_bits));
      }
      if (lane < kSelCluster) *cluster.map_shared_rank(&row_eq[i], lane) = n_eq;
    }
  cluster.sync();
  // exclusive prefix over the rows (one row per thread, nb <= 1024): rank of a row's first copy in row-major order
  unsigned int mine = tid < nb ? row_eq[tid] : 0u, incl = mine;
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  if (lane == 31) scan_tmp[warp] = incl;
  __syncthreads();
  unsigned int base = 0;
  for (int w = 0; w < warp; ++w) base += scan_tmp[w];
  __syncthreads();
  if (tid < nb) row_eq[tid] = base + incl - mine;
  __syncthreads();

  // marking: everything above the cut value, and the first k_eq copies of it in row-major order
  for (int i = row0; i < nb; i += kStride) {
    unsigned int rank0 = row_eq[i];
    for (int j0 = 0; j0 < nb; j0 += 32) {
      const int j = j0 + lane;
      const bool causal = j <= i;
      const unsigned int bits = causal ? score_bits(sc[(size_t)i * nb + j]) : 0u;
      const bool eq = causal && !cut.all && bits == cut.cut_bits;
      const unsigned int bal = __ballot_sync(0xffffffffu, eq);
      const bool on = causal && (cut.all || bits > cut.cut_bits || (eq && rank0 + __popc(bal & ((1u << lane) - 1u)) < cut.k_eq));
      if (j < nb) mk[(size_t)i * nb + j] = (uint8_t)(on ? 1 : 0);
      rank0 += __popc(bal);
    }
  }
  cluster.sync();      // nobody leaves while a neighbour may still read its shared memory
}

// ---- per row: force the diagonal into an empty row, compact the ascending list; one warp per row
__global__ void compact_rows_kernel(uint8_t* __restrict__ mask, int n_maps, int nb, int32_t* __restrict__ counts,
                                    int32_t* __restrict__ indices, const int32_t* __restrict__ active) {
  const int lane = threadIdx.x & 31;
  const long w = (long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (w >= (long)n_maps * nb) return;
  const int mp = (int)(w / nb), i = (int)(w % nb);
  if (active && active[mp] == 0) return;          // a map nobody will read
  uint8_t* row = mask + ((size_t)mp * nb + i) * nb;
  int32_t* irow = indices + ((size_t)mp * nb + i) * nb;
  int cnt = 0;
  for (int j0 = 0; j0 < nb; j0 += 32) {
    const int j = j0 + lane;
    const bool on = j <= i && row[j] != 0;
    const unsigned int bal = __ballot_sync(0xffffffffu, on);
    if (on) irow[cnt + __popc(bal & ((1u << lane) - 1u))] = j;
    cnt += __popc(bal);
  }
  if (cnt == 0) {                          // a row-block must keep at least one key-block: its diagonal
    if (lane == 0) { row[i] = 1; irow[0] = i; }
    cnt = 1;
  }
  __syncwarp();
  for (int j = cnt + lane; j < nb; j += 32) irow[j] = -1;
  if (lane == 0) counts[(size_t)mp * nb + i] = cnt;
}

// ---- "Determine Sparse Pattern" ---------------------------------------------------------------
// pooled last row: grid (Nb, n_heads), d threads.  Block j: mean of the last query block against the mean
// of key block j; the last block uses the visible half.
__global__ void last_row_pooled_kernel(const PooledArgs a) {
  __shared__ double red[4];
  const int j = blockIdx.x, slot = blockIdx.y, col = threadIdx.x;
  const int h = a.heads.v[slot], g = h / a.group;
  const int last = a.Nb - 1;
  const __nv_bfloat16* q = a.q + (size_t)h * a.q_sh + (size_t)last * a.B * a.q_sn + col;
  const __nv_bfloat16* k = a.k + (size_t)g * a.k_sh + (size_t)j * a.B * a.k_sn + col;
  double acc = 0.0, denom;
  if (j < last) {
    double qsum = 0.0, ksum = 0.0;
    for (int r = 0; r < a.B; ++r) {
      qsum += (double)__bfloat162float(q[(size_t)r * a.q_sn]);
      ksum += (double)__bfloat162float(k[(size_t)r * a.k_sn]);
    }
    acc = qsum * ksum;
    denom = (double)a.B * (double)a.B;
  } else {
    double kcum = 0.0;
    for (int r = 0; r < a.B; ++r) {
      kcum += (double)__bfloat162float(k[(size_t)r * a.k_sn]);
      acc = fma((double)__bfloat162float(q[(size_t)r * a.q_sn]), kcum, acc);
    }
    denom = 0.5 * (double)a.B * (double)(a.B + 1);
  }
  acc = warp_sum(acc);
  if ((col & 31) == 0) red[col >> 5] = acc;
  __syncthreads();
  if (col == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    a.pooled[(size_t)slot * a.Nb + j] = t * a.scale / denom;
  }
}

// one CTA of 256 threads per head: softmax of the pooled last row, the two Jensen-Shannon distances, the decision
__global__ void decide_pattern_kernel(const double* __restrict__ pooled_last, int nb, const float* __restrict__ pivot_rows,
                                      HeadTable row_of_head, float delta, float tau, int32_t* __restrict__ pattern,
                                      float* __restrict__ dist) {
  __shared__ double red[8];
  __shared__ double bc[2];
  const int slot = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double* z = pooled_last + (size_t)slot * nb;
  const int prow = row_of_head.v[slot];
  const float* at = prow >= 0 ? pivot_rows + (size_t)prow * nb : nullptr;
  auto block_reduce = [&](double v, bool is_max) {
    v = is_max ? warp_max(v) : warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    if (tid == 0) {
      double t = red[0];
      for (int w = 1; w < (int)(blockDim.x >> 5); ++w) t = is_max ? fmax(t, red[w]) : t + red[w];
      bc[0] = t;
    }
    __syncthreads();
    return bc[0];
  };
  double m = -CUDART_INF;
  for (int j = tid; j < nb; j += blockDim.x) m = fmax(m, z[j]);
  m = block_reduce(m, true);
  double s = 0.0;
  for (int j = tid; j < nb; j += blockDim.x) s += exp(z[j] - m);
  s = block_reduce(s, false);
  const double inv = 1.0 / s, u = 1.0 / (double)nb;
  // JSD(p || q) = 1/2 sum p ln(p/m) + 1/2 sum q ln(q/m), m = (p + q)/2, 0 ln 0 = 0
  double js_u = 0.0, js_a = 0.0;
  for (int j = tid; j < nb; j += blockDim.x) {
    const double p = exp(z[j] - m) * inv;
    {
      const double mm = 0.5 * (p + u);
      js_u += (p > 0.0 ? p * log(p / mm) : 0.0) + u * log(u / mm);
    }
    if (at) {
      const double q = (double)at[j], mm = 0.5 * (p + q);
      js_a += (p > 0.0 ? p * log(p / mm) : 0.0) + (q > 0.0 ? q * log(q / mm) : 0.0);
    }
  }
  js_u = block_reduce(js_u, false);
  js_a = block_reduce(js_a, false);
  if (tid == 0) {
    const float d_sparse = (float)sqrt(fmax(0.5 * js_u, 0.0));
    const float d_sim = at ? (float)sqrt(fmax(0.5 * js_a, 0.0)) : CUDART_INF_F;
    pattern[slot] = (d_sparse < delta && d_sim < tau) ? 0 : 1;
    if (dist) { dist[2 * slot] = d_sparse; dist[2 * slot + 1] = d_sim; }
  }
}

}  // namespace

size_t pooled_scratch_bytes(int n_heads, int Nb, int d) { return (size_t)n_heads * Nb * (2 * (size_t)d + 1) * sizeof(double); }

cudaError_t launch_pooled_logits(const PooledArgs& a, cudaStream_t s) {
  if (a.n_heads == 0) return cudaSuccess;
  block_means_kernel<<<dim3(a.Nb, a.n_heads), a.d, 0, s>>>(a);
  pooled_logits_kernel<<<dim3(a.Nb, a.n_heads), 128, 0, s>>>(a);
  return cudaGetLastError();
}

cudaError_t launch_pattern_from_pooled(const double* pooled, int n_maps, int nb, double gamma, float* scores,
                                       uint8_t* mask, int32_t* counts, int32_t* indices, float* last_row,
                                       cudaStream_t s) {
  if (n_maps == 0) return cudaSuccess;
  const long rows = (long)n_maps * nb;
  pooled_softmax_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, s>>>(pooled, n_maps, nb, scores, last_row);
  global_select_kernel<<<dim3(kSelCluster, n_maps), kSelThreads, 0, s>>>(scores, nb, gamma, mask);
  compact_rows_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, s>>>(mask, n_maps, nb, counts, indices, nullptr);
  return cudaGetLastError();
}

namespace {

// softmax of each row of z [n, nb] -> out; one CTA of 256 threads per row
__global__ void row_softmax_kernel(const double* __restrict__ z, int nb, float* __restrict__ out) {
  __shared__ double red[8];
  __shared__ double bc;
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double* in = z + (size_t)row * nb;
  double m = -CUDART_INF;
  for (int j = tid; j < nb; j += blockDim.x) m = fmax(m, in[j]);
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  if (tid == 0) { double t = red[0]; for (int w = 1; w < 8; ++w) t = fmax(t, red[w]); bc = t; }
  __syncthreads();
  m = bc;
  double s = 0.0;
  for (int j = tid; j < nb; j += blockDim.x) s += exp(in[j] - m);
  s = warp_sum(s);
  __syncthreads();
  if (lane == 0) red[warp] = s;
  __syncthreads();
  if (tid == 0) { double t = 0.0; for (int w = 0; w < 8; ++w) t += red[w]; bc = t; }
  __syncthreads();
  const double inv = 1.0 / bc;
  for (int j = tid; j < nb; j += blockDim.x) out[(size_t)row * nb + j] = (float)(exp(in[j] - m) * inv);
}

}  // namespace

cudaError_t launch_last_row_distribution(const PooledArgs& a, float* out, cudaStream_t s) {
  if (a.n_heads == 0) return cudaSuccess;
  last_row_pooled_kernel<<<dim3(a.Nb, a.n_heads), a.d, 0, s>>>(a);
  row_softmax_kernel<<<a.n_heads, 256, 0, s>>>(a.pooled, a.Nb, out);
  return cudaGetLastError();
}

namespace {
// decisions of "Determine Sparse Pattern" -> which list each member walks, which members need the
// vertical-slash search, pattern codes (0 dense, 1 shared pivot, 2 vertical-slash) and mask sources per head
__global__ void finalize_pattern_kernel(const int32_t* __restrict__ decide, HeadTable pivot_slot_of_member,
                                        HeadTable head_of_member, int n_members, HeadTable pivot_heads, int n_pivots,
                                        int32_t* __restrict__ lists_dev, int32_t* __restrict__ active,
                                        int32_t* __restrict__ pattern_out, int32_t* __restrict__ src_dev) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n_members) {
    const int ps = pivot_slot_of_member.v[t], h = head_of_member.v[t];
    int list, act, code;
    if (ps < 0) { list = -1; act = 0; code = 0; }                       // no pivotal pattern for its cluster: dense
    else if (decide[t] == 0) { list = ps; act = 0; code = 1; }          // shares the pivot's pattern
    else { list = n_pivots + t; act = 1; code = 2; }                    // falls back to its own vertical-slash pattern
    lists_dev[t] = list;
    active[t] = act;
    src_dev[h] = list;
    if (pattern_out) pattern_out[h] = code;
  } else if (t < n_members + n_pivots) {
    const int p = t - n_members, h = pivot_heads.v[p];
    src_dev[h] = p;
    if (pattern_out) pattern_out[h] = 0;
  }
}
}  // namespace

namespace {
// sqrt(JSD(a^ || uniform)) of each row of dist [n, nb]; one CTA of 256 threads per row
__global__ void js_uniform_kernel(const float* __restrict__ dist, int nb, float* __restrict__ d_sparse) {
  __shared__ double red[8];
  const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* p_ = dist + (size_t)row * nb;
  const double u = 1.0 / (double)nb;
  double js = 0.0;
  for (int j = tid; j < nb; j += blockDim.x) {
    const double p = (double)p_[j], mm = 0.5 * (p + u);
    js += (p > 0.0 ? p * log(p / mm) : 0.0) + u * log(u / mm);
  }
  js = warp_sum(js);
  if (lane == 0) red[warp] = js;
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    d_sparse[row] = (float)sqrt(fmax(0.5 * t, 0.0));
  }
}

// For each listed head: sqrt(JSD(a^_head || a~_slot)) < tau ?  decide = 0 (share) : 1.  Heads with slot < 0 get 1.
// a_hat [Hq, nb] indexed by head, a_tilde [n_slots, nb]; one CTA of 256 threads per listed head.
__global__ void js_pair_decide_kernel(const float* __restrict__ a_hat, const float* __restrict__ a_tilde, int nb,
                                      HeadTable heads, HeadTable slot_of, float tau, int32_t* __restrict__ decide) {
  __shared__ double red[8];
  const int t = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sl = slot_of.v[t];
  if (sl < 0) { if (tid == 0) decide[t] = 1; return; }
  const float* p_ = a_hat + (size_t)heads.v[t] * nb;
  const float* q_ = a_tilde + (size_t)sl * nb;
  double js = 0.0;
  for (int j = tid; j < nb; j += blockDim.x) {
    const double p = (double)p_[j], q = (double)q_[j], mm = 0.5 * (p + q);
    js += (p > 0.0 ? p * log(p / mm) : 0.0) + (q > 0.0 ? q * log(q / mm) : 0.0);
  }
  js = warp_sum(js);
  if (lane == 0) red[warp] = js;
  __syncthreads();
  if (tid == 0) {
    double s = 0.0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) s += red[w];
    decide[t] = (float)sqrt(fmax(0.5 * s, 0.0)) < tau ? 0 : 1;
  }
}

// lists / flags / codes of a layer driven by the cross-layer dictionary.  Member t: cand_slot >= 0 and decide == 0 ->
// it walks dictionary slot cand_slot (pattern 1); otherwise its own vertical-slash list vs_base + t (pattern 2).
__global__ void finalize_layer_kernel(const int32_t* __restrict__ decide, HeadTable cand_slot, HeadTable head_of_member,
                                      int n_members, HeadTable pivot_heads, HeadTable pivot_slots, int n_pivots, int vs_base,
                                      int32_t* __restrict__ lists_dev, int32_t* __restrict__ active,
                                      int32_t* __restrict__ pattern_out, int32_t* __restrict__ src_dev) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < n_members) {
    const int cs = cand_slot.v[t], h = head_of_member.v[t];
    const bool share = cs >= 0 && decide[t] == 0;
    const int list = share ? cs : vs_base + t;
    lists_dev[t] = list;
    active[t] = share ? 0 : 1;
    src_dev[h] = list;
    if (pattern_out) pattern_out[h] = share ? 1 : 2;
  } else if (t < n_members + n_pivots) {
    const int p = t - n_members, h = pivot_heads.v[p];
    src_dev[h] = pivot_slots.v[p];
    if (pattern_out) pattern_out[h] = 0;
  }
}
}  // namespace

cudaError_t launch_js_uniform(const float* dist, int n, int nb, float* d_sparse, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  js_uniform_kernel<<<n, 256, 0, s>>>(dist, nb, d_sparse);
  return cudaGetLastError();
}

cudaError_t launch_js_pair_decide(const float* a_hat, const float* a_tilde, int nb, const HeadTable& heads,
                                  const HeadTable& slot_of, int n, float tau, int32_t* decide, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  js_pair_decide_kernel<<<n, 256, 0, s>>>(a_hat, a_tilde, nb, heads, slot_of, tau, decide);
  return cudaGetLastError();
}

cudaError_t launch_finalize_layer(const int32_t* decide, const HeadTable& cand_slot, const HeadTable& head_of_member, int n_members,
                                  const HeadTable& pivot_heads, const HeadTable& pivot_slots, int n_pivots, int vs_base,
                                  int32_t* lists_dev, int32_t* active, int32_t* pattern_out, int32_t* src_dev, cudaStream_t s) {
  const int n = n_members + n_pivots;
  if (n == 0) return cudaSuccess;
  finalize_layer_kernel<<<(n + 127) / 128, 128, 0, s>>>(decide, cand_slot, head_of_member, n_members, pivot_heads, pivot_slots,
                                                        n_pivots, vs_base, lists_dev, active, pattern_out, src_dev);
  return cudaGetLastError();
}

cudaError_t launch_finalize_pattern(const int32_t* decide, const HeadTable& pivot_slot_of_member, const HeadTable& head_of_member,
                                    int n_members, const HeadTable& pivot_heads, int n_pivots, int32_t* lists_dev,
                                    int32_t* active, int32_t* pattern_out, int32_t* src_dev, cudaStream_t s) {
  const int n = n_members + n_pivots;
  if (n == 0) return cudaSuccess;
  finalize_pattern_kernel<<<(n + 127) / 128, 128, 0, s>>>(decide, pivot_slot_of_member, head_of_member, n_members, pivot_heads,
                                                          n_pivots, lists_dev, active, pattern_out, src_dev);
  return cudaGetLastError();
}

cudaError_t launch_compact_rows(uint8_t* mask, int n_maps, int nb, int32_t* counts, int32_t* indices, cudaStream_t s,
                                const int32_t* active) {
  const long rows = (long)n_maps * nb;
  if (rows == 0) return cudaSuccess;
  compact_rows_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, s>>>(mask, n_maps, nb, counts, indices, active);
  return cudaGetLastError();
}

cudaError_t launch_determine_pattern(const PooledArgs& a, const float* pivot_rows, const HeadTable& row_of_head,
                                     float delta, float tau, int32_t* pattern, float* dist, cudaStream_t s) {
  if (a.n_heads == 0) return cudaSuccess;
  last_row_pooled_kernel<<<dim3(a.Nb, a.n_heads), a.d, 0, s>>>(a);     // a.pooled: [n_heads, Nb] here
  decide_pattern_kernel<<<a.n_heads, 256, 0, s>>>(a.pooled, a.Nb, pivot_rows, row_of_head, delta, tau, pattern, dist);
  return cudaGetLastError();
}

}  // namespace sp
