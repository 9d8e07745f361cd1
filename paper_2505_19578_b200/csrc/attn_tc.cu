// Tensor-core attention kernel for sm_100a: dense (pivot) and block-sparse
// (member) causal attention in one template.
//
//   Section 5.1:  O = softmax(Q K^T / sqrt(d) - c (1 - M)) V,  c -> infinity,
//   causal.  A pivot walks every causal key-block and also emits the softmax
//   probability mass of each (query-block, key-block) tile; a member walks the
//   compacted list of key-blocks its cluster's pivot selected.
//
// One CTA owns one (head, query row-block).  Warp roles:
//   warps 0-3  softmax: thread t owns query row t = TMEM lane t.  Reads S from
//              TMEM, keeps the running max / sum, writes P (bf16) back into the
//              columns S occupied, rescales the O accumulator when the running
//              max moved, and runs the epilogue.
//   warp 4     producer: TMA loads of Q (once) and of one K and one V tile per
//              step into 128-byte-swizzled shared memory.
//   warp 5     MMA issuer: S = Q K^T (both operands from shared memory) and
//              O += P V (P from TMEM, V from shared memory, N-major), bf16 in,
//              fp32 accumulate in TMEM.  Owns the TMEM allocation.
// K and V have one shared-memory slot each: the K slot is free as soon as
// Q K^T has been read (long before the next step needs it), the V slot as soon
// as P V has.  Two CTAs share an SM, so one CTA's softmax overlaps the other's
// MMAs.
//
// Block importance in one pass: for each visited tile the softmax thread spills
// one float per row, stat = m + log2(sum_c 2^(s_c - m)) with m the row's running
// reference max at that step.  After the last tile the row's final log-sum-exp
// L is known and the tile mass is (1/B) sum_rows 2^(stat - L).
//
// Every wait on an mbarrier is bounded: when it runs out the CTA raises an abort
// flag, records SP_ERR_TIMEOUT in the status word, and all roles fall through
// to the common teardown (TMEM is freed, the kernel returns).
#include <mutex>

#include "tc_ptx.cuh"

namespace sp {
namespace {

using namespace tc;

constexpr int kThreads = 192;

// ------------------------------------------------------------------ shared-memory plan

template <int D, int BLK>
struct Plan {
  static constexpr int NBOX = D / 64;          // 64-column (128-byte) boxes per row
  static constexpr int QBOX = 128 * 128;       // bytes of one Q box: the MMA reads 128 rows
  static constexpr int KBOX = BLK * 128;       // bytes of one K / V box
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_OFF + NBOX * QBOX;
  static constexpr int V_OFF = K_OFF + NBOX * KBOX;
  static constexpr int MISC_OFF = V_OFF + NBOX * KBOX;
  static constexpr int MISC_BYTES = 1024;
  static constexpr int TOTAL = MISC_OFF + MISC_BYTES + 1024;   // + slack for 1024-byte alignment
  static constexpr int Q_TX = NBOX * BLK * 128;                 // bytes the Q loads deliver
  static constexpr int KV_TX = NBOX * KBOX;
  static constexpr int TMEM_COLS = (BLK + D) <= 128 ? 128 : 256;
  static constexpr int S_COL = 0;              // S (fp32, BLK columns); P (bf16 pairs) reuses its first BLK/2
  static constexpr int O_COL = BLK;            // O accumulator (fp32, D columns)
};

// barrier slots inside the MISC area
enum { BAR_Q_FULL = 0, BAR_K_FULL, BAR_V_FULL, BAR_QK_DONE, BAR_P_FULL, BAR_PV_DONE, BAR_COUNT };

template <int D, int BLK>
__global__ void __launch_bounds__(kThreads, 2)
attn_tc_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
               const __grid_constant__ CUtensorMap tm_v) {
  using P = Plan<D, BLK>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_u32(smem + P::Q_OFF), sK = smem_u32(smem + P::K_OFF), sV = smem_u32(smem + P::V_OFF);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + P::MISC_OFF);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + P::MISC_OFF + 64);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + P::MISC_OFF + 72);
  float* lse_smem = reinterpret_cast<float*>(smem + P::MISC_OFF + 128);   // 128 floats
  auto bar = [&](int which) { return smem_u32(bars + which); };

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i = a.Nb - 1 - (int)blockIdx.x;      // long row-blocks first
  const int slot = blockIdx.y;
  const int h = a.heads.v[slot];
  const int g = h / a.group;
  const int list = a.lists_dev ? a.lists_dev[slot] : a.lists.v[slot];   // decided on the device, or by the host
  int cnt = list >= 0 ? a.counts[(size_t)list * a.Nb + i] : i + 1;
  cnt = cnt < 0 ? 0 : (cnt > i + 1 ? i + 1 : cnt);
  const bool poisoned = *reinterpret_cast<volatile int*>(a.status) != 0;   // an earlier wait ran out: do no work
  if (poisoned) cnt = 0;
  const int32_t* idx = list >= 0 ? a.indices + ((size_t)list * a.Nb + i) * a.Nb : nullptr;
  const bool emit = a.importance != nullptr && list < 0;
  const Abort ab{abort_flag, a.status};
  // Optional phase trace (one CTA, one thread per role): {(event << 32) | tile, SM clock} pairs.
  const bool tracing = a.trace != nullptr && blockIdx.x == 0 && blockIdx.y == 0;
  int trace_n = 0;
  auto trace = [&](int role, int event, int tile) {
    if (tracing && trace_n < a.trace_cap) {
      long long* e = a.trace + ((size_t)role * a.trace_cap + trace_n) * 2;
      e[0] = ((long long)event << 32) | (unsigned)tile;
      e[1] = clock64();
      ++trace_n;
    }
  };

  if (threadIdx.x == 0) {
    mbar_init(bar(BAR_Q_FULL), 1);
    mbar_init(bar(BAR_K_FULL), 1);
    mbar_init(bar(BAR_V_FULL), 1);
    mbar_init(bar(BAR_QK_DONE), 1);
    mbar_init(bar(BAR_P_FULL), 128);
    mbar_init(bar(BAR_PV_DONE), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (BLK < 128) {
    // rows BLK..127 of the Q operand are never loaded: make them zeros
    for (int b = 0; b < P::NBOX; ++b) {
      uint4* z = reinterpret_cast<uint4*>(smem + P::Q_OFF + b * P::QBOX + BLK * 128);
      for (int x = threadIdx.x; x < (128 - BLK) * 128 / 16; x += kThreads) z[x] = make_uint4(0, 0, 0, 0);
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(smem_u32(tmem_slot), P::TMEM_COLS);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------------------ producer
    if (lane == 0 && cnt > 0) {
      mbar_expect_tx(bar(BAR_Q_FULL), P::Q_TX);
      for (int b = 0; b < P::NBOX; ++b) tma_load_3d(sQ + b * P::QBOX, &tm_q, bar(BAR_Q_FULL), b * 64, i * BLK, h);
      int issued_k = 0, issued_v = 0;
      bool ok = true;
      for (int t = 0; t < cnt && ok; ++t) {
        const int j = sp_in_range(idx ? idx[t] : t, 0, i, a.status, 60);
        if (t > 0) ok = mbar_wait(bar(BAR_QK_DONE), (t - 1) & 1, ab, 10);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_K_FULL), P::KV_TX);
        for (int b = 0; b < P::NBOX; ++b) tma_load_3d(sK + b * P::KBOX, &tm_k, bar(BAR_K_FULL), b * 64, j * BLK, g);
        ++issued_k;
        trace(0, 20, t);
        if (t > 0) ok = mbar_wait(bar(BAR_PV_DONE), (t - 1) & 1, ab, 11);
        if (!ok) break;
        mbar_expect_tx(bar(BAR_V_FULL), P::KV_TX);
        for (int b = 0; b < P::NBOX; ++b) tma_load_3d(sV + b * P::KBOX, &tm_v, bar(BAR_V_FULL), b * 64, j * BLK, g);
        ++issued_v;
        trace(0, 21, t);
      }
      if (*abort_flag) {
        // let the copies already in flight land before the CTA gives its shared memory back
        const long long t0 = clock64();
        while (clock64() - t0 < kWaitCycles / 8) {
          bool done = mbar_try_wait(bar(BAR_Q_FULL), 0);
          if (issued_k) done = done && mbar_try_wait(bar(BAR_K_FULL), (issued_k - 1) & 1);
          if (issued_v) done = done && mbar_try_wait(bar(BAR_V_FULL), (issued_v - 1) & 1);
          if (done) break;
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------------------ MMA issuer
    constexpr uint32_t idesc_qk = instr_desc(128, BLK, 0, 0);
    constexpr uint32_t idesc_pv = instr_desc(128, D, 0, 1);
    bool ok = cnt > 0 ? mbar_wait(bar(BAR_Q_FULL), 0, ab, 20) : false;
    for (int t = 0; t < cnt && ok; ++t) {
      ok = mbar_wait(bar(BAR_K_FULL), t & 1, ab, 21);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) {
        trace(1, 1, t);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
          const uint32_t off = (kk >> 2) * P::QBOX + (kk & 3) * 32;
          const uint32_t koff = (kk >> 2) * P::KBOX + (kk & 3) * 32;
          mma_ss(tmem + P::S_COL, smem_desc(sQ + off, 16, 1024), smem_desc(sK + koff, 16, 1024), idesc_qk, kk > 0);
        }
        mma_commit(bar(BAR_QK_DONE));
        trace(1, 2, t);
      }
      __syncwarp();
      ok = mbar_wait(bar(BAR_P_FULL), t & 1, ab, 22) && mbar_wait(bar(BAR_V_FULL), t & 1, ab, 23);
      if (!ok) break;
      tc_fence_after();
      if (lane == 0) {
        trace(1, 3, t);
#pragma unroll
        for (int kk = 0; kk < BLK / 16; ++kk) {
          // V tile: rows = keys (the MMA's K), 128-byte rows of 64 head-dim columns per box (N-major)
          mma_ts(tmem + P::O_COL, tmem + P::S_COL + kk * 8, smem_desc(sV + kk * 16 * 128, P::KBOX, 1024), idesc_pv,
                 (t > 0 || kk > 0) ? 1u : 0u);
        }
        mma_commit(bar(BAR_PV_DONE));
        trace(1, 4, t);
      }
      __syncwarp();
    }
  } else {
    // ------------------------------------------------------------ softmax + epilogue
    const int row = threadIdx.x;                       // TMEM lane == query row inside the tile
    const bool row_valid = row < BLK;
    const int r = i * BLK + (row_valid ? row : 0);
    const uint32_t tl = tmem + ((uint32_t)(warp * 32) << 16);
    const float scale = a.scale_log2;
    float* stats = emit ? a.tile_stats + ((size_t)slot * ((size_t)a.Nb * (a.Nb + 1) / 2) + (size_t)i * (i + 1) / 2) * BLK
                        : nullptr;
    float m_ref = -CUDART_INF_F, l = 0.f;
    bool ok = cnt > 0;
    for (int t = 0; t < cnt && ok; ++t) {
      const int j = sp_in_range(idx ? idx[t] : t, 0, i, a.status, 60);
      ok = mbar_wait(bar(BAR_QK_DONE), t & 1, ab, 30);
      if (!ok) break;
      tc_fence_after();
      if (threadIdx.x == 0) trace(2, 10, t);
      uint32_t s[BLK];
#pragma unroll
      for (int c = 0; c < BLK / 32; ++c) tmem_ld32(tl + P::S_COL + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
      if (threadIdx.x == 0) trace(2, 11, t);
      float mx = -CUDART_INF_F;
      if (j == i) {
#pragma unroll
        for (int c = 0; c < BLK; ++c) {
          float x = c > row ? -CUDART_INF_F : __uint_as_float(s[c]);
          s[c] = __float_as_uint(x);
          mx = fmaxf(mx, x);
        }
      } else {
#pragma unroll
        for (int c = 0; c < BLK; ++c) mx = fmaxf(mx, __uint_as_float(s[c]));
      }
      mx *= scale;
      if (threadIdx.x == 0) trace(2, 12, t);
      // the reference max only moves when the row max has grown by more than 2^8
      const float m_new = (mx > m_ref + 8.f) ? mx : m_ref;
      const float alpha = ex2_approx(m_ref - m_new);
      float sum = 0.f;
      uint32_t p[BLK / 2];
#pragma unroll
      for (int c = 0; c < BLK; c += 2) {
        const float p0 = ex2_approx(fmaf(__uint_as_float(s[c]), scale, -m_new));
        const float p1 = ex2_approx(fmaf(__uint_as_float(s[c + 1]), scale, -m_new));
        sum += p0 + p1;
        p[c / 2] = pack_bf16(p0, p1);
      }
      l = l * alpha + sum;
      if (threadIdx.x == 0) trace(2, 13, t);
      if (emit && row_valid) stats[(size_t)sp_in_range(t, 0, i, a.status, 61) * BLK + row] = m_new + log2f(sum);
      if (t > 0 && __any_sync(0xffffffffu, m_new != m_ref)) {
        // O of the previous steps is relative to the old reference: bring it to the new one
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          tmem_ld32(tl + P::O_COL + c * 32, o);
#pragma unroll
          for (int x = 0; x < 32; ++x) o[x] = __float_as_uint(__uint_as_float(o[x]) * alpha);
          tmem_st32(tl + P::O_COL + c * 32, o);
        }
      }
      m_ref = m_new;
      if (threadIdx.x == 0) trace(2, 14, t);
#pragma unroll
      for (int c = 0; c < BLK / 64; ++c) tmem_st32(tl + P::S_COL + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&p[c * 32]));
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(bar(BAR_P_FULL));
      if (threadIdx.x == 0) trace(2, 15, t);
    }
    if (ok) ok = mbar_wait(bar(BAR_PV_DONE), (cnt - 1) & 1, ab, 31);
    float lse2 = 0.f;
    if (ok) {
      tc_fence_after();
      const float inv_l = 1.f / l;
      __nv_bfloat16* orow = a.o + (size_t)h * a.o_sh + (size_t)r * a.o_sn;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        uint32_t o[32];
        tmem_ld32(tl + P::O_COL + c * 32, o);
        if (row_valid) {
          uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            uint4 u;
            u.x = pack_bf16(__uint_as_float(o[8 * x + 0]) * inv_l, __uint_as_float(o[8 * x + 1]) * inv_l);
            u.y = pack_bf16(__uint_as_float(o[8 * x + 2]) * inv_l, __uint_as_float(o[8 * x + 3]) * inv_l);
            u.z = pack_bf16(__uint_as_float(o[8 * x + 4]) * inv_l, __uint_as_float(o[8 * x + 5]) * inv_l);
            u.w = pack_bf16(__uint_as_float(o[8 * x + 6]) * inv_l, __uint_as_float(o[8 * x + 7]) * inv_l);
            dst[x] = u;
          }
        }
      }
      lse2 = m_ref + log2f(l);
      if (a.lse && row_valid) a.lse[(size_t)slot * a.N + r] = lse2 * 0.6931471805599453f;
    }
    if (emit) {
      lse_smem[row] = lse2;
      // the four softmax warps: statistics and lse visible to one another, and one common decision
      // (a thread whose wait ran out must not leave the others at a barrier)
      if (bar_and(1, 128, ok)) {
        float* imp_row = a.importance + ((size_t)slot * a.Nb + i) * a.Nb;
        for (int t = warp; t < cnt; t += 4) {
          float acc = 0.f;
          for (int rr = lane; rr < BLK; rr += 32) acc += exp2f(stats[(size_t)t * BLK + rr] - lse_smem[rr]);
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
          if (lane == 0) imp_row[t] = acc * (1.f / BLK);
        }
        for (int jz = i + 1 + (int)threadIdx.x; jz < a.Nb; jz += 128) imp_row[jz] = 0.f;
      }
    }
    if (ok) {
    } else if (cnt == 0 && row_valid && !poisoned) {
      // an empty list is outside the contract; leave defined output (zeros) rather than garbage
      __nv_bfloat16* orow = a.o + (size_t)h * a.o_sh + (size_t)r * a.o_sn;
      for (int x = 0; x < D / 8; ++x) reinterpret_cast<uint4*>(orow)[x] = make_uint4(0, 0, 0, 0);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem, P::TMEM_COLS);
  }
}

// ------------------------------------------------------------------ host side

template <int D, int BLK>
cudaError_t launch(const AttnArgs& a, cudaStream_t s) {
  using P = Plan<D, BLK>;
  CUtensorMap tq, tk, tv;
  if (!make_map(&tq, a.q, a.q_sh, a.q_sn, a.n_q_heads, a.N, D, BLK) ||
      !make_map(&tk, a.k, a.k_sh, a.k_sn, a.n_kv_heads, a.N, D, BLK) ||
      !make_map(&tv, a.v, a.v_sh, a.v_sn, a.n_kv_heads, a.N, D, BLK))
    return cudaErrorInvalidValue;
  // at most two CTAs per SM (their TMEM allocations must both fit in 512 columns)
  constexpr int smem = P::TOTAL > 100 * 1024 ? P::TOTAL : 100 * 1024;
  cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel<D, BLK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  attn_tc_kernel<D, BLK><<<dim3(a.Nb, a.n_heads), kThreads, smem, s>>>(a, tq, tk, tv);
  return cudaGetLastError();
}

}  // namespace

// ------------------------------------------------------------------ fixed-scratch variant
//
// Scratch for callers that cannot allocate: the per-tile softmax statistics of a
// dense pivot launch live in this file-scope array instead of a cudaMalloc'ed
// workspace, and so do the status word and the work counter of the launch.
// Every device that loads the library carries the array until the process exits.
// In host code `g_fixed_scratch` is only a handle for the runtime, not a device
// address: the address a kernel may use comes from cudaGetSymbolAddress, asked
// once per device with that device current.
static __device__ __align__(256) unsigned char g_fixed_scratch[kFixedScratchBytes];
static __device__ __align__(256) int g_fixed_status[4];   // {code, where, work counter, unused}

namespace {
constexpr int kMaxDevices = 64;
void* g_fixed_scratch_addr[kMaxDevices];
void* g_fixed_status_addr[kMaxDevices];
bool g_fixed_ready[kMaxDevices];
std::mutex g_fixed_mutex;

// first call on this device (the caller made it current): resolve both symbols
cudaError_t fixed_setup(int device) {
  if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_fixed_mutex);
  if (g_fixed_ready[device]) return cudaSuccess;
  void* scratch = nullptr;
  void* status = nullptr;
  cudaError_t e = cudaGetSymbolAddress(&scratch, g_fixed_scratch);
  if (e != cudaSuccess) return e;
  e = cudaGetSymbolAddress(&status, g_fixed_status);
  if (e != cudaSuccess) return e;
  g_fixed_scratch_addr[device] = scratch;
  g_fixed_status_addr[device] = status;
  g_fixed_ready[device] = true;
  return cudaSuccess;
}
}  // namespace

// Bytes of the fixed array a launch needs (with the launch's device current).
size_t fixed_scratch_need(const AttnArgs& a) {
  if (!a.importance) return 0;
  return attn_pair_supported(a) ? attn_pair_stats_bytes(a.n_heads, a.Nb)
                                : (size_t)a.n_heads * tile_stats_bytes_per_head(a.Nb, a.B);
}

cudaError_t launch_attn_fixed_scratch(AttnArgs a, int device, cudaStream_t s) {
  cudaError_t e = fixed_setup(device);
  if (e != cudaSuccess) return e;
  if (fixed_scratch_need(a) > kFixedScratchBytes) return cudaErrorInvalidValue;
  a.tile_stats = static_cast<float*>(g_fixed_scratch_addr[device]);
  a.status = static_cast<int*>(g_fixed_status_addr[device]);
  a.work_counter = a.status + 2;
  // the status word keeps the previous call's value and the kernels refuse to work
  // when it is non-zero: it has to start at zero (the paired launch clears its work
  // counter itself).  The statistics need no clearing: every entry that is read has
  // been written by the same launch.
  e = cudaMemsetAsync(a.status, 0, 2 * sizeof(int), s);
  if (e != cudaSuccess) return e;
  return attn_pair_supported(a) ? launch_attn_pair(a, s) : launch_attn_tc(a, s);
}

// Reads the fixed status word of `device` back (and clears it when it is set).  The caller has synchronised.
cudaError_t fixed_status_read(int device, int* code, int* where) {
  cudaError_t e = fixed_setup(device);
  if (e != cudaSuccess) return e;
  int host[2] = {0, 0};
  e = cudaMemcpy(host, g_fixed_status_addr[device], sizeof(host), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return e;
  if (host[0] != 0) {
    e = cudaMemset(g_fixed_status_addr[device], 0, sizeof(host));
    if (e != cudaSuccess) return e;
  }
  if (code) *code = host[0];
  if (where) *where = host[1];
  return cudaSuccess;
}

cudaError_t launch_attn_tc(const AttnArgs& a, cudaStream_t s) {
  if (a.d == 128 && a.B == 128) return launch<128, 128>(a, s);
  if (a.d == 128 && a.B == 64) return launch<128, 64>(a, s);
  if (a.d == 64 && a.B == 128) return launch<64, 128>(a, s);
  if (a.d == 64 && a.B == 64) return launch<64, 64>(a, s);
  return cudaErrorInvalidValue;
}

namespace {
// One warp waits, with the given cycle limit, on an mbarrier that nothing ever arrives at: the wait runs out, the
// status word gets SP_ERR_TIMEOUT and the location id, and the kernel returns normally.
__global__ void wait_selftest_kernel(int* status, long long limit_cycles, int where) {
  __shared__ uint64_t bar_storage;
  __shared__ int abort_storage;
  const uint32_t bar = tc::smem_u32(&bar_storage);
  if (threadIdx.x == 0) {
    tc::mbar_init(bar, 1);
    abort_storage = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (*reinterpret_cast<volatile int*>(status) != 0) return;   // poisoned by an earlier failure: do no work, as every kernel here
  const tc::Abort ab{&abort_storage, status};
  tc::mbar_wait(bar, 0, ab, where, limit_cycles);
}
}  // namespace

cudaError_t launch_wait_selftest(int* status, long long limit_cycles, int where, cudaStream_t s) {
  wait_selftest_kernel<<<1, 32, 0, s>>>(status, limit_cycles, where);
  return cudaGetLastError();
}

}  // namespace sp
