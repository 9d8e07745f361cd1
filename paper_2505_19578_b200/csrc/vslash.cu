// Vertical-slash pattern search (Algorithm "Search Vertical Slash Pattern").
//
//   A^ = softmax(Q^ K^T / sqrt(d)) for a subset Q^ of the queries (here: the last
//   block), causal; a_v = its sums per key column, a_s = its sums per offset
//   o = query - key (the "slash" lines), both normalised; each is sorted and cut
//   at the minimum budget whose scores reach gamma; the union of the selected
//   lines becomes the mask.
//
// Q^ K^T is a dense 128 x N x 128 contraction per head: tcgen05 MMAs, K tiles by
// TMA, S in TMEM (two buffers, so the MMA of the next tile runs while this one is
// consumed).  Two sweeps over the keys, each split into chunks of key-blocks
// across CTAs:
//   sweep 0  D = Q^ K^T  (lane = query row): running max / sum per row and chunk;
//            a small kernel merges the chunks into the row's log-sum-exp.
//   sweep 1  D = K Q^^T  (lane = key, the operands swapped), so that a thread owns
//            one key column: p = exp(s - lse) down the column gives a_v directly
//            (one writer per key), and the slash sums go through a 255-entry window
//            in shared memory in 2^-40 fixed point (integer adds commute: the
//            result does not depend on the order of arrival) that slides along with
//            the key-blocks of a chunk; finished offsets are stored, and only the
//            two ends of a chunk are added atomically to global 64-bit counters.
// Then two cumulative cuts over vectors of N scores (select.cuh: exact
// fixed-point sums, ties to the smaller index), and the lines are turned into a
// block mask: block (i, j), j <= i, is computed if key-block j holds a selected
// column or a selected offset lies in [(i-j)B - (B-1), (i-j)B + (B-1)].
//
// Every wait on an mbarrier is bounded (see tc_ptx.cuh).
#include <cooperative_groups.h>
#include <math.h>
#include <string.h>

#include "select.cuh"
#include "tc_ptx.cuh"

namespace sp {
namespace {

using namespace tc;

constexpr int D = 128, BLK = 128;
constexpr int kVsThreads = 192;            // warps 0-3 consume S, warp 4 TMA producer, warp 5 MMA issuer
constexpr int kBox = 128 * 128, kTile = 2 * kBox;
constexpr int kVsQOff = 0, kVsKOff = kTile, kVsMiscOff = 3 * kTile;
constexpr int kVsSmem = kVsMiscOff + 4096 + 1024;
constexpr double kSlashFix = 1099511627776.0;   // 2^40

enum { VB_Q = 0, VB_K_FULL, VB_K_EMPTY = VB_K_FULL + 2, VB_S_FULL = VB_K_EMPTY + 2, VB_S_EMPTY = VB_S_FULL + 2, VB_COUNT = VB_S_EMPTY + 2 };

struct VsArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  int64_t q_sh, q_sn, k_sh, k_sn;
  int n_q_heads, n_kv_heads, group, N, Nb, n_heads, chunk;   // chunk: key-blocks per CTA
  HeadTable heads;
  float scale_log2;
  float2* partial;               // [n_heads, n_chunks, 128]: (max, sum) per row and chunk, log2 domain
  float* lse2;                   // [n_heads, 128]
  float* a_v;                    // [n_heads, N]
  unsigned long long* a_s_fx;    // [n_heads, N], 2^-40 fixed point
  const int32_t* active;
  int* status;
};

template <int SWEEP>
__global__ void __launch_bounds__(kVsThreads, 2)
vs_sweep_kernel(const VsArgs a, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem + kVsQOff), sK = smem_u32(smem + kVsKOff);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + kVsMiscOff);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + kVsMiscOff + 128);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + kVsMiscOff + 132);
  float* lse_smem = reinterpret_cast<float*>(smem + kVsMiscOff + 256);                       // [128]
  unsigned long long* window = reinterpret_cast<unsigned long long*>(smem + kVsMiscOff + 1024);  // [256]
  auto bar = [&](int which) { return smem_u32(bars + which); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int chunk = blockIdx.x, slot = blockIdx.y;
  const int h = a.heads.v[slot], g = h / a.group;
  const int j0 = chunk * a.chunk;
  int n_tiles = a.Nb - j0 < a.chunk ? a.Nb - j0 : a.chunk;
  if (*reinterpret_cast<volatile int*>(a.status) != 0) n_tiles = 0;     // an earlier wait ran out: do no work
  if (a.active && a.active[slot] == 0) n_tiles = 0;                      // head not selected for the search
  const int last = a.Nb - 1;
  const Abort ab{abort_flag, a.status};

  if (threadIdx.x == 0) {
    mbar_init(bar(VB_Q), 1);
    for (int s = 0; s < 2; ++s) {
      mbar_init(bar(VB_K_FULL + s), 1);
      mbar_init(bar(VB_K_EMPTY + s), 1);
      mbar_init(bar(VB_S_FULL + s), 1);
      mbar_init(bar(VB_S_EMPTY + s), 128);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (SWEEP == 1 && threadIdx.x < 128) lse_smem[threadIdx.x] = a.lse2[(size_t)slot * 128 + threadIdx.x];
  if (SWEEP == 1) for (int x = threadIdx.x; x < 256; x += kVsThreads) window[x] = 0ull;
  if (warp == 5) tmem_alloc(smem_u32(tmem_slot), 256);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------ producer
    if (lane == 0 && n_tiles > 0) {
      mbar_expect_tx(bar(VB_Q), kTile);
      for (int b = 0; b < 2; ++b) tma_load_3d(sQ + b * kBox, &tm_q, bar(VB_Q), b * 64, last * BLK, h);
      int issued = 0;
      bool ok = true;
      for (int t = 0; t < n_tiles && ok; ++t) {
        const int st = t & 1;
        if (t >= 2) ok = mbar_wait(bar(VB_K_EMPTY + st), ((t >> 1) - 1) & 1, ab, 40);
        if (!ok) break;
        mbar_expect_tx(bar(VB_K_FULL + st), kTile);
        for (int b = 0; b < 2; ++b) tma_load_3d(sK + st * kTile + b * kBox, &tm_k, bar(VB_K_FULL + st), b * 64, (j0 + t) * BLK, g);
        ++issued;
      }
      if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < kWaitCycles / 8) {
          bool done = mbar_try_wait(bar(VB_Q), 0);
          for (int back = 1; back <= 2; ++back) {
            const int m = issued - back;
            if (m >= 0) done = done && mbar_try_wait(bar(VB_K_FULL + (m & 1)), (m >> 1) & 1);
          }
          if (done) break;
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc = instr_desc(128, 128, 0, 0);
    const uint64_t dq0 = smem_desc(sQ, 16, 1024), dk0 = smem_desc(sK, 16, 1024);
    bool ok = n_tiles > 0 ? mbar_wait(bar(VB_Q), 0, ab, 41) : false;
    for (int t = 0; t < n_tiles && ok; ++t) {
      const int st = t & 1;
      ok = mbar_wait(bar(VB_K_FULL + st), (t >> 1) & 1, ab, 42);
      if (ok && t >= 2) ok = mbar_wait(bar(VB_S_EMPTY + st), ((t >> 1) - 1) & 1, ab, 43);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) {
        const uint64_t dk = dk0 + (uint64_t)((st * kTile) >> 4);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = ((kk >> 2) * kBox + (kk & 3) * 32) >> 4;
          // sweep 0: S = Q^ K^T (lane = query); sweep 1: S^T = K Q^^T (lane = key)
          if (SWEEP == 0) mma_ss(tmem + st * 128, dq0 + off, dk + off, idesc, kk > 0);
          else mma_ss(tmem + st * 128, dk + off, dq0 + off, idesc, kk > 0);
        }
        mma_commit(bar(VB_S_FULL + st));
        mma_commit(bar(VB_K_EMPTY + st));
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ consumers: thread = TMEM lane
    const int x = threadIdx.x;                          // sweep 0: query row; sweep 1: key inside the tile
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
    const float scale = a.scale_log2;
    float m = -CUDART_INF_F, l = 0.f;
    bool ok = true;
    // Every thread runs every iteration (a thread whose wait ran out only skips the work), so that
    // nobody is left alone at the named barriers of sweep 1.
    for (int t = 0; t < n_tiles; ++t) {
      const int st = t & 1, j = j0 + t;
      if (ok) ok = mbar_wait(bar(VB_S_FULL + st), (t >> 1) & 1, ab, 44);
      if (ok) {
        tc_fence_after();
        if (SWEEP == 0) {
          // running max and sum of the row over this tile's keys, 32 at a time (the last key-block is
          // the diagonal one; key 0 of a tile is visible to every row, so m is finite from the first
          // chunk on and a fully masked later chunk leaves it alone)
#pragma unroll 1
          for (int c0 = 0; c0 < BLK; c0 += 32) {
            uint32_t s[32];
            tmem_ld32(tl + st * 128 + c0, s);
            float cm = -CUDART_INF_F;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              float v = __uint_as_float(s[e]) * scale;
              if (j == last && c0 + e > x) v = -CUDART_INF_F;
              s[e] = __float_as_uint(v);
              cm = fmaxf(cm, v);
            }
            const float m_new = fmaxf(m, cm);
            float sum = 0.f;
#pragma unroll
            for (int e = 0; e < 32; ++e) sum += ex2_approx(__uint_as_float(s[e]) - m_new);
            l = l * ex2_approx(m - m_new) + sum;
            m = m_new;
          }
        } else {
          // this thread's key against the 128 queries: p = 2^(s - lse) where the key is visible
          const int c_glob = j * BLK + x;
          float colsum = 0.f;
#pragma unroll 1
          for (int r0 = 0; r0 < BLK; r0 += 32) {
            uint32_t s[32];
            tmem_ld32(tl + st * 128 + r0, s);
#pragma unroll
            for (int e = 0; e < 32; ++e) {
              const int r = r0 + e;
              float p = ex2_approx(fmaf(__uint_as_float(s[e]), scale, -lse_smem[r]));
              if (j == last && x > r) p = 0.f;
              colsum += p;
              // offset o = (N - 128 + r) - c_glob lives at window index r - x + 127
              atomicAdd(&window[r - x + 127], (unsigned long long)__float2ull_rn(p * (float)kSlashFix));
            }
          }
          a.a_v[(size_t)slot * a.N + c_glob] = colsum;
        }
        tc_fence_before();
        mbar_arrive(bar(VB_S_EMPTY + st));
      }
      if (SWEEP == 1) {
        // The window covers offsets o_base .. o_base + 254 and moves down by 128 with every key-block: its
        // upper 128 entries are final once this tile is in (they also hold the previous tile's share, carried
        // over below) and are written out; its lower 127 entries are carried to the next tile.  Only the ends of
        // a chunk meet another CTA's tiles and need atomic adds.
        asm volatile("bar.sync 1, 128;" ::: "memory");
        const long o_base = (long)(a.N - BLK) - (long)j * BLK - 127;
        unsigned long long* dst = a.a_s_fx + (size_t)slot * a.N;
        {
          const int idx = 127 + x;
          const unsigned long long wv = window[idx];
          const long o = o_base + idx;
          if (o >= 0 && o < a.N) {
            if (t == 0) { if (wv != 0ull) atomicAdd(&dst[o], wv); }
            else dst[o] = wv;
          }
        }
        const unsigned long long carry = x < 127 ? window[x] : 0ull;
        if (t == n_tiles - 1 && x < 127) {
          const long o = o_base + x;
          if (carry != 0ull && o >= 0 && o < a.N) atomicAdd(&dst[o], carry);
        }
        asm volatile("bar.sync 1, 128;" ::: "memory");
        window[x] = 0ull;
        if (x < 127) window[x + 128] = (t == n_tiles - 1) ? 0ull : carry;
        asm volatile("bar.sync 1, 128;" ::: "memory");
      }
    }
    if (SWEEP == 0 && ok && n_tiles > 0) a.partial[((size_t)slot * gridDim.x + chunk) * 128 + x] = make_float2(m, l);
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, 256);
  }
}

// merge the chunks' (max, sum) into the row's log2-sum-exp; one CTA per head, thread = row
__global__ void vs_lse_kernel(const float2* __restrict__ partial, int n_chunks, float* __restrict__ lse2) {
  const int slot = blockIdx.x, r = threadIdx.x;
  float m = -CUDART_INF_F;
  for (int c = 0; c < n_chunks; ++c) m = fmaxf(m, partial[((size_t)slot * n_chunks + c) * 128 + r].x);
  float l = 0.f;
  for (int c = 0; c < n_chunks; ++c) {
    const float2 p = partial[((size_t)slot * n_chunks + c) * 128 + r];
    l += p.y * exp2f(p.x - m);
  }
  lse2[(size_t)slot * 128 + r] = m + log2f(l);
}

__global__ void vs_slash_to_float_kernel(const unsigned long long* __restrict__ fx, long n, float* __restrict__ out) {
  const long e = (long)blockIdx.x * blockDim.x + threadIdx.x;
  if (e < n) out[e] = (float)((double)fx[e] * (1.0 / kSlashFix));
}

// ---- cumulative cut over a vector: minimum descending prefix whose normalised scores reach gamma --------
// A cluster of 4 CTAs per vector, each owning a contiguous quarter; block sums are widened to the cluster
// through distributed shared memory (every CTA adds the four partial sums in the same order).
constexpr int kSelThreads = 1024;
constexpr int kVecCluster = 4;

// grid = (kVecCluster, n_vectors); vector v at scores + v * n
__global__ void __cluster_dims__(kVecCluster, 1, 1) __launch_bounds__(kSelThreads)
vector_select_kernel(const float* __restrict__ scores, long n, double gamma, uint8_t* __restrict__ sel,
                     const int32_t* __restrict__ active) {
  if (active && active[blockIdx.y] == 0) return;           // the whole cluster returns: nobody waits for anybody
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ unsigned long long sh_sum[kSelThreads / 32 + 1];
  __shared__ unsigned long long partial[2];
  __shared__ unsigned int eq_total[kVecCluster];            // copies of the cut value in each CTA's quarter
  __shared__ unsigned int warp_cnt[kSelThreads / 32];
  __shared__ unsigned int running;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, rank = (int)cluster.block_rank();
  const float* sc = scores + (size_t)blockIdx.y * n;
  uint8_t* out = sel + (size_t)blockIdx.y * n;
  const long per = (n + kVecCluster - 1) / kVecCluster;
  const long lo = rank * per, hi = lo + per < n ? lo + per : n;
  auto for_each = [&](auto f) {
    for (long e = lo + tid; e < hi; e += kSelThreads) f(sc[e]);
  };
  int pass = 0;
  auto widen = [&](unsigned long long x) {
    const int buf = pass & 1;
    ++pass;
    if (tid == 0) partial[buf] = x;
    cluster.sync();
    unsigned long long t = 0;
    for (int r = 0; r < kVecCluster; ++r) t += *cluster.map_shared_rank(&partial[buf], r);
    return t;
  };
  const CutResult cut = block_cumulative_cut<kSelThreads>(for_each, widen, gamma, sh_sum);

  // copies of the cut value in the quarters before this one
  unsigned int n_eq = 0;
  if (!cut.all)
    for (long e = lo + tid; e < hi; e += kSelThreads) n_eq += score_bits(sc[e]) == cut.cut_bits;
  n_eq = (unsigned int)block_sum_u64<kSelThreads>(n_eq, sh_sum);
  if (tid < kVecCluster) *cluster.map_shared_rank(&eq_total[rank], tid) = n_eq;
  cluster.sync();
  if (tid == 0) {
    unsigned int t = 0;
    for (int r = 0; r < rank; ++r) t += eq_total[r];
    running = t;
  }
  __syncthreads();
  // ordered marking: above the cut value, and its first k_eq copies by index
  for (long base = lo; base < hi; base += kSelThreads) {
    const long e = base + tid;
    const unsigned int bits = e < hi ? score_bits(sc[e]) : 0u;
    const bool eq = e < hi && !cut.all && bits == cut.cut_bits;
    const unsigned int bal = __ballot_sync(0xffffffffu, eq);
    if (lane == 0) warp_cnt[warp] = __popc(bal);
    __syncthreads();
    unsigned int before = running;
    for (int w = 0; w < warp; ++w) before += warp_cnt[w];
    const unsigned int rk = before + __popc(bal & ((1u << lane) - 1u));
    if (e < hi) out[e] = (uint8_t)((cut.all || bits > cut.cut_bits || (eq && rk < cut.k_eq)) ? 1 : 0);
    __syncthreads();
    if (tid == 0) {
      unsigned int t = 0;
      for (int w = 0; w < kSelThreads / 32; ++w) t += warp_cnt[w];
      running += t;
    }
    __syncthreads();
  }
  cluster.sync();      // nobody leaves while a neighbour may still read its shared memory
}

// ---- selected lines -> block mask; one CTA per head ----------------------------------------------------
__global__ void vs_lines_to_mask_kernel(const uint8_t* __restrict__ sel_v, const uint8_t* __restrict__ sel_s, int N, int nb,
                                        uint8_t* __restrict__ mask, const int32_t* __restrict__ active) {
  __shared__ uint8_t vb[kMaxNb], sb[kMaxNb];
  const int slot = blockIdx.x;
  if (active && active[slot] == 0) return;
  const uint8_t* sv = sel_v + (size_t)slot * N;
  const uint8_t* ss = sel_s + (size_t)slot * N;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, n_warps = blockDim.x >> 5;
  for (int j = warp; j < nb; j += n_warps) {
    bool any_v = false, any_s = false;
    for (int c = lane; c < BLK; c += 32) any_v |= sv[(size_t)j * BLK + c] != 0;
    // block offset j: slash offsets j*B - (B-1) .. j*B + (B-1)
    for (int o = j * BLK - (BLK - 1) + lane; o <= j * BLK + (BLK - 1); o += 32)
      if (o >= 0 && o < N) any_s |= ss[o] != 0;
    any_v = __any_sync(0xffffffffu, any_v);
    any_s = __any_sync(0xffffffffu, any_s);
    if (lane == 0) { vb[j] = any_v; sb[j] = any_s; }
  }
  __syncthreads();
  uint8_t* m = mask + (size_t)slot * nb * nb;
  for (int i = warp; i < nb; i += n_warps)
    for (int j = lane; j < nb; j += 32) m[(size_t)i * nb + j] = (uint8_t)((j <= i && (vb[j] || sb[i - j])) ? 1 : 0);
}

}  // namespace

size_t vslash_scratch_bytes(int n_heads, int N, int chunk) {
  const int Nb = N / BLK, n_chunks = (Nb + chunk - 1) / chunk;
  size_t b = 0;
  b += (size_t)n_heads * n_chunks * 128 * sizeof(float2);
  b += (size_t)n_heads * 128 * sizeof(float);
  b += 2 * (size_t)n_heads * N * sizeof(float);                 // a_v, a_s
  b += (size_t)n_heads * N * sizeof(unsigned long long);
  b += 2 * (size_t)n_heads * N;                                 // sel_v, sel_s
  return b + 5 * 256;
}

cudaError_t launch_vertical_slash(const VslashArgs& v, cudaStream_t s) {
  if (v.n_heads == 0) return cudaSuccess;
  if (v.d != D || v.B != BLK) return cudaErrorInvalidValue;
  const int Nb = v.N / BLK, chunk = v.chunk, n_chunks = (Nb + chunk - 1) / chunk;
  auto up = [](size_t x) { return (x + 255) / 256 * 256; };
  char* p = static_cast<char*>(v.scratch);
  VsArgs a;
  memset(&a, 0, sizeof(a));
  a.partial = reinterpret_cast<float2*>(p); p += up((size_t)v.n_heads * n_chunks * 128 * sizeof(float2));
  a.lse2 = reinterpret_cast<float*>(p);     p += up((size_t)v.n_heads * 128 * sizeof(float));
  a.a_v = reinterpret_cast<float*>(p);      p += up((size_t)v.n_heads * v.N * sizeof(float));
  float* a_s = reinterpret_cast<float*>(p); p += up((size_t)v.n_heads * v.N * sizeof(float));
  a.a_s_fx = reinterpret_cast<unsigned long long*>(p); p += up((size_t)v.n_heads * v.N * sizeof(unsigned long long));
  uint8_t* sel = reinterpret_cast<uint8_t*>(p);                 // [2][n_heads][N]: the scores a_v | a_s are contiguous too
  a.q = v.q; a.k = v.k; a.q_sh = v.q_sh; a.q_sn = v.q_sn; a.k_sh = v.k_sh; a.k_sn = v.k_sn;
  a.n_q_heads = v.n_q_heads; a.n_kv_heads = v.n_kv_heads; a.group = v.n_q_heads / v.n_kv_heads;
  a.N = v.N; a.Nb = Nb; a.n_heads = v.n_heads; a.chunk = chunk; a.heads = v.heads;
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)D));
  a.status = v.status;
  a.active = v.active;
  CUtensorMap tq, tk;
  if (!make_map(&tq, a.q, a.q_sh, a.q_sn, a.n_q_heads, a.N, D, BLK) ||
      !make_map(&tk, a.k, a.k_sh, a.k_sn, a.n_kv_heads, a.N, D, BLK))
    return cudaErrorInvalidValue;
  cudaError_t e;
  if ((e = cudaFuncSetAttribute(vs_sweep_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kVsSmem)) != cudaSuccess) return e;
  if ((e = cudaFuncSetAttribute(vs_sweep_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kVsSmem)) != cudaSuccess) return e;
  if ((e = cudaMemsetAsync(a.a_s_fx, 0, (size_t)v.n_heads * v.N * sizeof(unsigned long long), s)) != cudaSuccess) return e;
  vs_sweep_kernel<0><<<dim3(n_chunks, v.n_heads), kVsThreads, kVsSmem, s>>>(a, tq, tk);
  vs_lse_kernel<<<v.n_heads, 128, 0, s>>>(a.partial, n_chunks, a.lse2);
  vs_sweep_kernel<1><<<dim3(n_chunks, v.n_heads), kVsThreads, kVsSmem, s>>>(a, tq, tk);
  const long n_all = (long)v.n_heads * v.N;
  vs_slash_to_float_kernel<<<(unsigned)((n_all + 255) / 256), 256, 0, s>>>(a.a_s_fx, n_all, a_s);
  // a_v and a_s are adjacent: 2 * n_heads vectors of N scores (up() keeps them adjacent when n_heads * N * 4 is a multiple of 256)
  vector_select_kernel<<<dim3(kVecCluster, v.n_heads), kSelThreads, 0, s>>>(a.a_v, v.N, v.gamma, sel, v.active);
  vector_select_kernel<<<dim3(kVecCluster, v.n_heads), kSelThreads, 0, s>>>(a_s, v.N, v.gamma, sel + (size_t)v.n_heads * v.N, v.active);
  vs_lines_to_mask_kernel<<<v.n_heads, 512, 0, s>>>(sel, sel + (size_t)v.n_heads * v.N, v.N, Nb, v.mask, v.active);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  if (v.sel_v_out) {
    if ((e = cudaMemcpyAsync(v.sel_v_out, sel, (size_t)v.n_heads * v.N, cudaMemcpyDeviceToDevice, s)) != cudaSuccess) return e;
  }
  if (v.sel_s_out) {
    if ((e = cudaMemcpyAsync(v.sel_s_out, sel + (size_t)v.n_heads * v.N, (size_t)v.n_heads * v.N, cudaMemcpyDeviceToDevice, s)) != cudaSuccess) return e;
  }
  return launch_compact_rows(v.mask, v.n_heads, Nb, v.counts, v.indices, s, v.active);
}

}  // namespace sp
