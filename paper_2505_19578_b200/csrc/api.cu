// Host side of the C ABI: argument validation, workspace carving, the sharing
// table (Algorithm "Share Pivotal Pattern") and the launch sequence of
// sp_prefill_attn (Algorithm "Sparse Attention" with the pattern decision fixed
// by the caller).  No arithmetic of the method happens on the host.
#include <math.h>
#include <string.h>

#include <new>
#include <vector>

#include "common.cuh"

struct sp_ctx {
  int device = 0;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int* status = nullptr;  // device int[4]: {code, where, work counter of the paired kernel, unused}
  int kernel = 0;         // 0 tensor-core (paired where supported), 1 CUDA-core cross-check, 2 tensor-core single-tile
  int64_t launches = 0;
  long long* trace = nullptr;  // caller's device buffer for the phase trace, or null
  int trace_cap = 0;
  // sp_prefill_attn_host: device copies of q, k, v, out (+ masks) and the copy streams
  void* stage = nullptr;
  size_t stage_bytes = 0;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  std::vector<cudaEvent_t> events;
};

// Cross-layer dictionary of pivotal patterns: cluster id -> (mask, compacted lists, representative a~).
// List slots 0..C-1 belong to the clusters, slots C..C+H-1 are scratch for the vertical-slash lists of a layer.
struct sp_pattern_dict {
  int device = 0;
  int C = 0, H = 0, Nb = 0, B = 0;
  int64_t N = 0;
  void* buf = nullptr;
  uint8_t* masks = nullptr;
  int32_t* counts = nullptr;
  int32_t* indices = nullptr;
  float* a_tilde = nullptr;
  std::vector<char> has;
};

namespace {

using namespace sp;

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    target = dev;
  }
  ~DeviceGuard() {
    if (prev >= 0 && prev != target) cudaSetDevice(prev);
  }
  int target = -1;
};

size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Problem {
  int Hq, Hkv, N, d, B, Nb;
};

int check_tensor(const sp_tensor* t) {
  if (!t || !t->data) return SP_ERR_INVALID_ARG;
  for (int x = 0; x < 4; ++x)
    if (t->shape[x] <= 0) return SP_ERR_INVALID_ARG;
  if (t->stride[3] != 1) return SP_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(t->data) & 15) != 0) return SP_ERR_INVALID_ARG;
  for (int x = 0; x < 3; ++x)
    if (t->stride[x] < 0 || (t->stride[x] % 8) != 0) return SP_ERR_INVALID_ARG;
  // a broadcast view (stride 0 over heads or rows, e.g. an expanded K) would make the tensor maps address memory
  // past the caller's buffer: refuse it
  for (int x = 1; x < 3; ++x)
    if (t->stride[x] == 0 && t->shape[x] > 1) return SP_ERR_INVALID_ARG;
  if (t->stride[2] < t->shape[3]) return SP_ERR_INVALID_ARG;
  return SP_OK;
}

int check_problem(const sp_tensor* q, const sp_tensor* k, const sp_tensor* v, const sp_tensor* out, int block,
                  Problem* p) {
  int rc;
  if ((rc = check_tensor(q)) || (rc = check_tensor(k)) || (rc = check_tensor(v)) || (rc = check_tensor(out))) return rc;
  for (int x = 0; x < 4; ++x) {
    if (k->shape[x] != v->shape[x]) return SP_ERR_INVALID_ARG;
    if (q->shape[x] != out->shape[x]) return SP_ERR_INVALID_ARG;
  }
  if (q->shape[2] != k->shape[2] || q->shape[3] != k->shape[3]) return SP_ERR_INVALID_ARG;
  if (q->shape[0] != k->shape[0]) return SP_ERR_INVALID_ARG;
  if (q->shape[0] != 1) return SP_ERR_UNSUPPORTED;
  const int64_t Hq = q->shape[1], Hkv = k->shape[1], N = q->shape[2], d = q->shape[3];
  if (Hq > kMaxHeads) return SP_ERR_UNSUPPORTED;
  if (Hq % Hkv != 0) return SP_ERR_UNSUPPORTED;
  if (d != 64 && d != 128) return SP_ERR_UNSUPPORTED;
  if (block != 64 && block != 128) return SP_ERR_UNSUPPORTED;
  if (N % block != 0) return SP_ERR_UNSUPPORTED;
  if (N / block > kMaxNb) return SP_ERR_UNSUPPORTED;
  p->Hq = (int)Hq; p->Hkv = (int)Hkv; p->N = (int)N; p->d = (int)d; p->B = block; p->Nb = (int)(N / block);
  return SP_OK;
}

AttnArgs base_args(const sp_ctx* ctx, const Problem& p, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                   const sp_tensor* out) {
  AttnArgs a;
  memset(&a, 0, sizeof(a));
  a.q = static_cast<const __nv_bfloat16*>(q->data);
  a.k = static_cast<const __nv_bfloat16*>(k->data);
  a.v = static_cast<const __nv_bfloat16*>(v->data);
  a.o = static_cast<__nv_bfloat16*>(out->data);
  a.q_sh = q->stride[1]; a.q_sn = q->stride[2];
  a.k_sh = k->stride[1]; a.k_sn = k->stride[2];
  a.v_sh = v->stride[1]; a.v_sn = v->stride[2];
  a.o_sh = out->stride[1]; a.o_sn = out->stride[2];
  a.n_q_heads = p.Hq; a.n_kv_heads = p.Hkv;
  a.N = p.N; a.d = p.d; a.B = p.B; a.Nb = p.Nb; a.group = p.Hq / p.Hkv;
  a.status = ctx->status;
  a.work_counter = ctx->status ? ctx->status + 2 : nullptr;
  a.trace = ctx->trace;
  a.trace_cap = ctx->trace_cap;
  a.pair_heads = ctx->kernel != 3;
  a.scale_log2 = (float)(1.4426950408889634 / sqrt((double)p.d));
  return a;
}

int reserve(sp_ctx* ctx, size_t bytes) {
  if (bytes <= ctx->ws_bytes) return SP_OK;
  if (ctx->ws) {
    if (cudaDeviceSynchronize() != cudaSuccess) return SP_ERR_CUDA;
    cudaFree(ctx->ws);
    ctx->ws = nullptr;
    ctx->ws_bytes = 0;
  }
  void* p = nullptr;
  if (cudaMalloc(&p, bytes) != cudaSuccess) {
    cudaGetLastError();
    return SP_ERR_WORKSPACE;
  }
  ctx->ws = p;
  ctx->ws_bytes = bytes;
  return SP_OK;
}

int launch_attn(sp_ctx* ctx, const AttnArgs& a, cudaStream_t s) {
  if (a.n_heads == 0) return SP_OK;
  cudaError_t e;
  if (ctx->kernel == 1) e = launch_attn_simt(a, s);
  else if ((ctx->kernel == 0 || ctx->kernel == 3) && attn_pair_supported(a)) e = launch_attn_pair(a, s);
  else e = launch_attn_tc(a, s);
  if (e != cudaSuccess) return SP_ERR_CUDA;
  ctx->launches += 1;
  return SP_OK;
}

// Bytes of tile statistics a dense launch over n_heads heads with importance needs.  `paired`: the launch goes to the
// paired kernel (one region per CTA, used by every launch in turn); otherwise one region per head.
bool goes_paired(int kernel, int d, int B) { return (kernel == 0 || kernel == 3) && d == 128 && B == 128; }
size_t stats_bytes(bool paired, int n_heads, int Nb, int B) {
  return paired ? attn_pair_stats_bytes(n_heads, Nb) : (size_t)n_heads * tile_stats_bytes_per_head(Nb, B);
}

struct WsLayout {
  size_t imp, mask, counts, indices, stats, total;
};

WsLayout ws_layout(int Nb, int B, int n_pivots, bool paired) {
  WsLayout w;
  size_t off = 0;
  const size_t nn = (size_t)Nb * Nb;
  w.imp = off;     off += align_up(n_pivots * nn * sizeof(float));
  w.mask = off;    off += align_up(n_pivots * nn);
  w.counts = off;  off += align_up((size_t)n_pivots * Nb * sizeof(int32_t));
  w.indices = off; off += align_up(n_pivots * nn * sizeof(int32_t));
  w.stats = off;   off += align_up(stats_bytes(paired, n_pivots, Nb, B));
  w.total = off;
  return w;
}

// Workspace of sp_prefill_attn_auto and of sp_prefill_attn_layer (offsets in bytes, each 256-byte aligned).
struct AutoLayout {
  size_t imp, scores, mask, counts, indices, scratch, atilde, rows, small, vs, total;
};
AutoLayout auto_layout(const Problem& p, int n_pivots, int n_members, bool pooled, bool paired) {
  AutoLayout w;
  const size_t nn = (size_t)p.Nb * p.Nb;
  const int lists = n_pivots + n_members;
  const int rows = n_pivots > n_members ? n_pivots : n_members;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  w.imp = take(n_pivots * nn * (pooled ? sizeof(double) : sizeof(float)));   // importance, or the pooled map
  w.scores = take(pooled ? n_pivots * nn * sizeof(float) : 0);
  w.mask = take(lists * nn);
  w.counts = take((size_t)lists * p.Nb * sizeof(int32_t));
  w.indices = take(lists * nn * sizeof(int32_t));
  w.scratch = take(pooled ? pooled_scratch_bytes(n_pivots, p.Nb, p.d) : stats_bytes(paired, n_pivots, p.Nb, p.B));
  w.atilde = take((size_t)n_pivots * p.Nb * sizeof(float));
  w.rows = take((size_t)rows * p.Nb * sizeof(double));
  w.small = take((size_t)(3 * kMaxHeads + p.Hq) * sizeof(int32_t));
  w.vs = take(vslash_scratch_bytes(n_members, p.N, 8));
  w.total = off;
  return w;
}
struct LayerLayout {
  size_t ahat, rows, small, imp, scores, scratch, vs, total;
};
LayerLayout layer_layout(const Problem& p, int n_new_max, bool pooled, bool paired) {
  LayerLayout w;
  const size_t nn = (size_t)p.Nb * p.Nb;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += align_up(bytes); return o; };
  w.ahat = take((size_t)p.Hq * p.Nb * sizeof(float));
  w.rows = take((size_t)p.Hq * p.Nb * sizeof(double));
  w.small = take((size_t)(4 * kMaxHeads) * sizeof(int32_t) + (size_t)kMaxHeads * sizeof(float));
  w.imp = take(n_new_max * nn * (pooled ? sizeof(double) : sizeof(float)));
  w.scores = take(pooled ? nn * sizeof(float) : 0);
  w.scratch = take(pooled ? pooled_scratch_bytes(n_new_max, p.Nb, p.d) : stats_bytes(paired, n_new_max, p.Nb, p.B));
  w.vs = take(vslash_scratch_bytes(p.Hq, p.N, 8));
  w.total = off;
  return w;
}

__global__ void gather_masks_kernel(const uint8_t* __restrict__ pivot_masks, HeadTable src, int nb,
                                    uint8_t* __restrict__ out, const int32_t* __restrict__ src_dev = nullptr) {
  const int i = blockIdx.x, h = blockIdx.y;
  const int s = src_dev ? src_dev[h] : src.v[h];
  uint8_t* dst = out + ((size_t)h * nb + i) * nb;
  if (s >= 0) {
    const uint8_t* from = pivot_masks + ((size_t)s * nb + i) * nb;
    for (int j = threadIdx.x; j < nb; j += blockDim.x) dst[j] = from[j];
  } else {
    for (int j = threadIdx.x; j < nb; j += blockDim.x) dst[j] = j <= i ? 1 : 0;
  }
}

}  // namespace

extern "C" {

const char* sp_strerror(int code) {
  switch (code) {
    case SP_OK: return "ok";
    case SP_ERR_INVALID_ARG: return "invalid argument";
    case SP_ERR_UNSUPPORTED: return "unsupported size or layout";
    case SP_ERR_WORKSPACE: return "workspace allocation failed";
    case SP_ERR_CUDA: return "CUDA call failed";
    case SP_ERR_TIMEOUT: return "device-side wait timed out";
    case SP_ERR_SCRATCH_LIMIT: return "problem needs more scratch than the library's fixed scratch array holds";
    case SP_ERR_RANGE: return "an index left its range (range-checked debug build)";
    default: return "unknown error code";
  }
}

int sp_ctx_create(sp_ctx** out, int device) {
  if (!out) return SP_ERR_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess) { cudaGetLastError(); return SP_ERR_CUDA; }
  if (device < 0 || device >= n) return SP_ERR_INVALID_ARG;
  DeviceGuard g(device);
  if (!g.ok) return SP_ERR_CUDA;
  sp_ctx* c = new (std::nothrow) sp_ctx();
  if (!c) return SP_ERR_WORKSPACE;
  c->device = device;
  if (cudaMalloc(&c->status, 4 * sizeof(int)) != cudaSuccess || cudaMemset(c->status, 0, 4 * sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    delete c;
    return SP_ERR_CUDA;
  }
  *out = c;
  return SP_OK;
}

int sp_ctx_destroy(sp_ctx* ctx) {
  if (!ctx) return SP_OK;
  DeviceGuard g(ctx->device);
  if (ctx->ws) cudaFree(ctx->ws);
  if (ctx->status) cudaFree(ctx->status);
  if (ctx->stage) cudaFree(ctx->stage);
  if (ctx->s_in) cudaStreamDestroy(ctx->s_in);
  if (ctx->s_out) cudaStreamDestroy(ctx->s_out);
  for (cudaEvent_t e : ctx->events) cudaEventDestroy(e);
  delete ctx;
  return SP_OK;
}

int sp_workspace_bytes(int64_t seq, int n_q_heads, int n_kv_heads, int head_dim, int block, int n_pivots,
                       size_t* bytes) {
  if (!bytes || seq <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || n_pivots < 0) return SP_ERR_INVALID_ARG;
  if (block != 64 && block != 128) return SP_ERR_UNSUPPORTED;
  if (head_dim != 64 && head_dim != 128) return SP_ERR_UNSUPPORTED;
  if (seq % block != 0 || seq / block > kMaxNb || n_q_heads % n_kv_heads != 0) return SP_ERR_UNSUPPORTED;
  *bytes = ws_layout((int)(seq / block), block, n_pivots, goes_paired(0, head_dim, block)).total;
  return SP_OK;
}

int sp_workspace_bytes_patterns(int64_t seq, int n_q_heads, int n_kv_heads, int head_dim, int block, int n_pivots,
                                int pooled_construction, size_t* auto_bytes, size_t* layer_bytes) {
  if (seq <= 0 || n_q_heads <= 0 || n_kv_heads <= 0 || n_pivots < 0 || n_pivots > n_q_heads) return SP_ERR_INVALID_ARG;
  if (head_dim != 128 || block != 128) return SP_ERR_UNSUPPORTED;
  if (seq % block != 0 || seq / block > kMaxNb || n_q_heads % n_kv_heads != 0 || n_q_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  Problem p{n_q_heads, n_kv_heads, (int)seq, head_dim, block, (int)(seq / block)};
  if (auto_bytes) *auto_bytes = auto_layout(p, n_pivots, n_q_heads - n_pivots, pooled_construction != 0, true).total;
  if (layer_bytes) *layer_bytes = layer_layout(p, n_pivots, pooled_construction != 0, true).total;
  return SP_OK;
}

int sp_ctx_reserve(sp_ctx* ctx, size_t bytes) {
  if (!ctx) return SP_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  return reserve(ctx, bytes);
}

int sp_get_status(sp_ctx* ctx, int* code, int* where) {
  if (!ctx) return SP_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  int host[2] = {0, 0};
  if (cudaMemcpy(host, ctx->status, sizeof(host), cudaMemcpyDeviceToHost) != cudaSuccess) return SP_ERR_CUDA;
  if (host[0] != 0 && cudaMemset(ctx->status, 0, sizeof(host)) != cudaSuccess) return SP_ERR_CUDA;
  if (code) *code = host[0];
  if (where) *where = host[1];
  return SP_OK;
}

int sp_selftest_wait_timeout(sp_ctx* ctx, int64_t limit_cycles, void* stream) {
  if (!ctx || limit_cycles <= 0 || limit_cycles > 2000000000ll) return SP_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  if (launch_wait_selftest(ctx->status, (long long)limit_cycles, 99, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SP_ERR_CUDA;
  ctx->launches += 1;
  return SP_OK;
}

int sp_ctx_set_kernel(sp_ctx* ctx, int which) {
  if (!ctx || which < 0 || which > 3) return SP_ERR_INVALID_ARG;
  ctx->kernel = which;
  return SP_OK;
}

int64_t sp_ctx_launch_count(const sp_ctx* ctx) { return ctx ? ctx->launches : 0; }

int sp_internal_pair_work_order(const int32_t* heads, const int32_t* lists, int n_heads, int n_q_heads, int n_kv_heads,
                                int n_row_blocks, int n_sm, int pair_heads, int32_t* tiles_out, int* n_groups_out) {
  if (!heads || !lists || !tiles_out || n_heads <= 0 || n_heads > kMaxHeads || n_q_heads <= 0 || n_kv_heads <= 0 ||
      n_q_heads % n_kv_heads != 0 || n_row_blocks <= 0 || n_sm <= 0)
    return SP_ERR_INVALID_ARG;
  AttnArgs a;
  memset(&a, 0, sizeof(a));
  a.n_heads = n_heads; a.n_q_heads = n_q_heads; a.n_kv_heads = n_kv_heads; a.group = n_q_heads / n_kv_heads;
  a.Nb = n_row_blocks; a.pair_heads = pair_heads;
  for (int t = 0; t < n_heads; ++t) {
    if (heads[t] < 0 || heads[t] >= n_q_heads) return SP_ERR_INVALID_ARG;
    a.heads.v[t] = heads[t];
    a.lists.v[t] = lists[t];
  }
  attn_pair_work_order(a, n_sm);
  const int n_items = n_heads * ((n_row_blocks + 1) / 2);
  for (int raw = 0; raw < n_items; ++raw) {
    int sa, ra, sb, rb;
    if (!attn_pair_item(a, raw, &sa, &ra, &sb, &rb)) return SP_ERR_INVALID_ARG;
    tiles_out[4 * raw + 0] = sa; tiles_out[4 * raw + 1] = ra; tiles_out[4 * raw + 2] = sb; tiles_out[4 * raw + 3] = rb;
  }
  if (n_groups_out) *n_groups_out = a.n_groups;
  return SP_OK;
}

int sp_ctx_set_trace(sp_ctx* ctx, int64_t* events, int events_per_role) {
  if (!ctx || events_per_role < 0 || (events_per_role > 0 && !events)) return SP_ERR_INVALID_ARG;
  ctx->trace = events_per_role > 0 ? reinterpret_cast<long long*>(events) : nullptr;
  ctx->trace_cap = events_per_role;
  return SP_OK;
}

int sp_dense_pivot_attn(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v, const int32_t* heads,
                        int n_heads, int block, sp_tensor* out, float* importance_out, float* lse_out, void* stream) {
  if (!ctx || !heads || n_heads < 0) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, v, out, block, &p);
  if (rc) return rc;
  if (n_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  for (int t = 0; t < n_heads; ++t)
    if (heads[t] < 0 || heads[t] >= p.Hq) return SP_ERR_INVALID_ARG;
  if (n_heads == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  AttnArgs a = base_args(ctx, p, q, k, v, out);
  a.n_heads = n_heads;
  for (int t = 0; t < n_heads; ++t) { a.heads.v[t] = heads[t]; a.lists.v[t] = -1; }
  a.importance = importance_out;
  a.lse = lse_out;
  if (importance_out && ctx->kernel != 1) {
    if ((rc = reserve(ctx, align_up(stats_bytes(goes_paired(ctx->kernel, p.d, p.B), n_heads, p.Nb, p.B))))) return rc;
    a.tile_stats = static_cast<float*>(ctx->ws);
  }
  return launch_attn(ctx, a, static_cast<cudaStream_t>(stream));
}

int sp_dense_pivot_attn_fixed_scratch(int device, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                                      const int32_t* heads, int n_heads, int block, sp_tensor* out,
                                      float* importance_out, float* lse_out, void* stream) {
  if (!heads || n_heads < 0) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, v, out, block, &p);
  if (rc) return rc;
  if (n_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  for (int t = 0; t < n_heads; ++t)
    if (heads[t] < 0 || heads[t] >= p.Hq) return SP_ERR_INVALID_ARG;
  if (n_heads == 0) return SP_OK;
  DeviceGuard g(device);
  if (!g.ok) return SP_ERR_CUDA;
  sp_ctx no_ctx;                       // only so that base_args has somewhere to read a status pointer from
  AttnArgs a = base_args(&no_ctx, p, q, k, v, out);
  a.n_heads = n_heads;
  for (int t = 0; t < n_heads; ++t) { a.heads.v[t] = heads[t]; a.lists.v[t] = -1; }
  a.importance = importance_out;
  a.lse = lse_out;
  if (fixed_scratch_need(a) > kFixedScratchBytes) return SP_ERR_SCRATCH_LIMIT;
  if (launch_attn_fixed_scratch(a, device, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SP_ERR_CUDA;
  return SP_OK;
}

int sp_fixed_scratch_status(int device, int* code, int* where) {
  DeviceGuard g(device);
  if (!g.ok) return SP_ERR_CUDA;
  if (fixed_status_read(device, code, where) != cudaSuccess) { cudaGetLastError(); return SP_ERR_CUDA; }
  return SP_OK;
}

int sp_block_mask_from_importance(sp_ctx* ctx, const float* importance, int n_maps, int nb, float gamma,
                                  uint8_t* mask_out, int32_t* counts_out, int32_t* indices_out, void* stream) {
  if (!ctx || !importance || !counts_out || !indices_out || n_maps < 0 || nb <= 0) return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f)) return SP_ERR_INVALID_ARG;
  if (nb > kMaxNb) return SP_ERR_UNSUPPORTED;
  if (n_maps == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  MaskArgs m{importance, n_maps, nb, (double)gamma, mask_out, counts_out, indices_out};
  if (launch_block_mask(m, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SP_ERR_CUDA;
  ctx->launches += 1;
  return SP_OK;
}

int sp_block_sparse_attn(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v, const int32_t* heads,
                         int n_heads, const int32_t* list_of_head, const int32_t* counts, const int32_t* indices,
                         int n_lists, int block, sp_tensor* out, void* stream) {
  if (!ctx || !heads || !list_of_head || n_heads < 0 || n_lists < 0) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, v, out, block, &p);
  if (rc) return rc;
  if (n_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  bool any_list = false;
  for (int t = 0; t < n_heads; ++t) {
    if (heads[t] < 0 || heads[t] >= p.Hq) return SP_ERR_INVALID_ARG;
    if (list_of_head[t] >= n_lists) return SP_ERR_INVALID_ARG;
    any_list |= list_of_head[t] >= 0;
  }
  if (any_list && (!counts || !indices)) return SP_ERR_INVALID_ARG;
  if (n_heads == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  AttnArgs a = base_args(ctx, p, q, k, v, out);
  a.n_heads = n_heads;
  for (int t = 0; t < n_heads; ++t) { a.heads.v[t] = heads[t]; a.lists.v[t] = list_of_head[t] < 0 ? -1 : list_of_head[t]; }
  a.counts = counts;
  a.indices = indices;
  return launch_attn(ctx, a, static_cast<cudaStream_t>(stream));
}

int sp_prefill_attn(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                    const int32_t* cluster_map, const int32_t* pivot_heads, int n_pivots, float gamma, int block,
                    sp_tensor* out, uint8_t* mask_out, void* stream) {
  if (!ctx || !cluster_map || n_pivots < 0 || (n_pivots > 0 && !pivot_heads)) return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f)) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, v, out, block, &p);
  if (rc) return rc;
  if (n_pivots > p.Hq) return SP_ERR_INVALID_ARG;

  // Sharing table: pivot slot of each cluster = first listed pivot belonging to it.
  int pivot_slot_of_head[kMaxHeads];
  for (int h = 0; h < p.Hq; ++h) pivot_slot_of_head[h] = -1;
  for (int t = 0; t < n_pivots; ++t) {
    const int h = pivot_heads[t];
    if (h < 0 || h >= p.Hq || pivot_slot_of_head[h] >= 0) return SP_ERR_INVALID_ARG;  // range / duplicate
    pivot_slot_of_head[h] = t;
  }
  auto cluster_pivot = [&](int c) {
    if (c < 0) return -1;
    for (int t = 0; t < n_pivots; ++t)
      if (cluster_map[pivot_heads[t]] == c) return t;
    return -1;
  };

  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const WsLayout w = ws_layout(p.Nb, p.B, n_pivots, goes_paired(ctx->kernel, p.d, p.B));
  if ((rc = reserve(ctx, w.total))) return rc;
  char* ws = static_cast<char*>(ctx->ws);
  float* imp = reinterpret_cast<float*>(ws + w.imp);
  uint8_t* pmask = reinterpret_cast<uint8_t*>(ws + w.mask);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + w.counts);
  int32_t* indices = reinterpret_cast<int32_t*>(ws + w.indices);
  float* stats = reinterpret_cast<float*>(ws + w.stats);

  // 1. pivots: dense + importance
  AttnArgs a = base_args(ctx, p, q, k, v, out);
  a.n_heads = n_pivots;
  for (int t = 0; t < n_pivots; ++t) { a.heads.v[t] = pivot_heads[t]; a.lists.v[t] = -1; }
  a.importance = imp;
  a.tile_stats = stats;
  if ((rc = launch_attn(ctx, a, s))) return rc;

  // 2. importance -> masks and lists
  if (n_pivots > 0) {
    MaskArgs m{imp, n_pivots, p.Nb, (double)gamma, pmask, counts, indices};
    if (launch_block_mask(m, s) != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 1;
  }

  // 3. everyone else: the cluster pivot's list, or dense when there is none
  AttnArgs b = base_args(ctx, p, q, k, v, out);
  b.counts = counts;
  b.indices = indices;
  HeadTable mask_src;
  int nb_heads = 0;
  for (int h = 0; h < p.Hq; ++h) {
    if (pivot_slot_of_head[h] >= 0) { mask_src.v[h] = pivot_slot_of_head[h]; continue; }
    const int t = cluster_pivot(cluster_map[h]);
    mask_src.v[h] = t;
    b.heads.v[nb_heads] = h;
    b.lists.v[nb_heads] = t;
    ++nb_heads;
  }
  b.n_heads = nb_heads;
  if ((rc = launch_attn(ctx, b, s))) return rc;

  if (mask_out) {
    gather_masks_kernel<<<dim3(p.Nb, p.Hq), 128, 0, s>>>(pmask, mask_src, p.Nb, mask_out);
    if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 1;
  }
  return SP_OK;
}

int sp_prefill_attn_host(sp_ctx* ctx, const void* q_host, const void* k_host, const void* v_host, int n_q_heads,
                         int n_kv_heads, int64_t seq, int head_dim, const int32_t* cluster_map,
                         const int32_t* pivot_heads, int n_pivots, float gamma, int block, void* out_host,
                         uint8_t* mask_out_host, void* stream) {
  if (!ctx || !q_host || !k_host || !v_host || !out_host || !cluster_map || n_pivots < 0 || (n_pivots > 0 && !pivot_heads))
    return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f) || n_q_heads <= 0 || n_kv_heads <= 0 || seq <= 0) return SP_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;

  // device copies: q | k | v | out | masks, each 256-byte aligned
  const size_t head_bytes = (size_t)seq * head_dim * sizeof(__nv_bfloat16);
  const size_t q_bytes = align_up((size_t)n_q_heads * head_bytes), kv_bytes = align_up((size_t)n_kv_heads * head_bytes);
  const int64_t nb = block > 0 ? seq / block : 0;
  const size_t mask_bytes = mask_out_host ? align_up((size_t)n_q_heads * nb * nb) : 0;
  const size_t need = 2 * q_bytes + 2 * kv_bytes + mask_bytes;
  sp_tensor q, k, v, o;
  auto view = [&](sp_tensor* t, void* data, int heads) {
    t->data = data;
    t->shape[0] = 1; t->shape[1] = heads; t->shape[2] = seq; t->shape[3] = head_dim;
    t->stride[0] = 0; t->stride[1] = seq * head_dim; t->stride[2] = head_dim; t->stride[3] = 1;
  };
  // validate sizes before anything is allocated (data pointers are placeholders here)
  view(&q, ctx, n_q_heads); view(&k, ctx, n_kv_heads); view(&v, ctx, n_kv_heads); view(&o, ctx, n_q_heads);
  {
    sp_tensor qa = q, ka = k, va = v, oa = o;
    qa.data = ka.data = va.data = oa.data = reinterpret_cast<void*>(uintptr_t(256));
    Problem chk;
    int rc = check_problem(&qa, &ka, &va, &oa, block, &chk);
    if (rc) return rc;
  }
  if (n_pivots > n_q_heads) return SP_ERR_INVALID_ARG;
  int pivot_slot_of_head[kMaxHeads];
  for (int h = 0; h < n_q_heads; ++h) pivot_slot_of_head[h] = -1;
  for (int t = 0; t < n_pivots; ++t) {
    const int h = pivot_heads[t];
    if (h < 0 || h >= n_q_heads || pivot_slot_of_head[h] >= 0) return SP_ERR_INVALID_ARG;
    pivot_slot_of_head[h] = t;
  }
  auto cluster_pivot = [&](int c) {
    if (c < 0) return -1;
    for (int t = 0; t < n_pivots; ++t)
      if (cluster_map[pivot_heads[t]] == c) return t;
    return -1;
  };

  if (need > ctx->stage_bytes) {
    if (ctx->stage) {
      if (cudaDeviceSynchronize() != cudaSuccess) return SP_ERR_CUDA;
      cudaFree(ctx->stage);
      ctx->stage = nullptr;
      ctx->stage_bytes = 0;
    }
    if (cudaMalloc(&ctx->stage, need) != cudaSuccess) { cudaGetLastError(); return SP_ERR_WORKSPACE; }
    ctx->stage_bytes = need;
  }
  if (!ctx->s_in && cudaStreamCreateWithFlags(&ctx->s_in, cudaStreamNonBlocking) != cudaSuccess) return SP_ERR_CUDA;
  if (!ctx->s_out && cudaStreamCreateWithFlags(&ctx->s_out, cudaStreamNonBlocking) != cudaSuccess) return SP_ERR_CUDA;
  size_t next_event = 0;
  auto event = [&]() -> cudaEvent_t {
    if (next_event == ctx->events.size()) {
      cudaEvent_t e = nullptr;
      if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return nullptr;
      ctx->events.push_back(e);
    }
    return ctx->events[next_event++];
  };
  // record on `from`, make `to` wait
  auto hand_over = [&](cudaStream_t from, cudaStream_t to) {
    cudaEvent_t e = event();
    return e && cudaEventRecord(e, from) == cudaSuccess && cudaStreamWaitEvent(to, e, 0) == cudaSuccess;
  };

  char* base = static_cast<char*>(ctx->stage);
  char* dq = base; char* dk = dq + q_bytes; char* dv = dk + kv_bytes; char* dout = dv + kv_bytes;
  uint8_t* dmask = mask_out_host ? reinterpret_cast<uint8_t*>(dout + q_bytes) : nullptr;
  view(&q, dq, n_q_heads); view(&k, dk, n_kv_heads); view(&v, dv, n_kv_heads); view(&o, dout, n_q_heads);
  Problem p;
  int rc = check_problem(&q, &k, &v, &o, block, &p);
  if (rc) return rc;
  const bool paired = goes_paired(ctx->kernel, p.d, p.B);
  const WsLayout w = ws_layout(p.Nb, p.B, n_pivots, paired);
  if ((rc = reserve(ctx, w.total))) return rc;
  char* ws = static_cast<char*>(ctx->ws);
  float* imp = reinterpret_cast<float*>(ws + w.imp);
  uint8_t* pmask = reinterpret_cast<uint8_t*>(ws + w.mask);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + w.counts);
  int32_t* indices = reinterpret_cast<int32_t*>(ws + w.indices);
  float* stats = reinterpret_cast<float*>(ws + w.stats);

  cudaStream_t sc = static_cast<cudaStream_t>(stream), sin = ctx->s_in, sout = ctx->s_out;
  const char* hq = static_cast<const char*>(q_host);
  char* ho = static_cast<char*>(out_host);
  auto copy_in_head = [&](int h) {
    return cudaMemcpyAsync(dq + (size_t)h * head_bytes, hq + (size_t)h * head_bytes, head_bytes, cudaMemcpyHostToDevice, sin) == cudaSuccess;
  };
  auto copy_out_head = [&](int h) {
    return cudaMemcpyAsync(ho + (size_t)h * head_bytes, dout + (size_t)h * head_bytes, head_bytes, cudaMemcpyDeviceToHost, sout) == cudaSuccess;
  };

  // The copy streams start after whatever the caller's stream already holds (an earlier call on
  // this context may still be reading the device copies).
  if (!hand_over(sc, sin) || !hand_over(sc, sout)) return SP_ERR_CUDA;

  // Order of the work (and, with it, of the copies in): cluster by cluster, the pivots one cluster ahead.  For a
  // pivot: its KV head (if not yet on the device) and its queries in, step 1 and step 2 for it alone, its output out;
  // for its cluster's members, in groups of one or two heads: their KV heads and queries in, step 4, outputs out.
  // Sequence: pivot 0, pivot 1, members 0, pivot 2, members 1, ..., members n-2, members n-1.  The copies in are the
  // longest resource of the call (1.6 GB against 1.1 GB out and 25 ms of kernels at 128K with 32 query heads; with the
  // copies out running beside them they take 32 ms), so the call cannot end before they do; what has to be kept short
  // is what follows the last copy in, and the copies out must have work from early on.  With every pivot first they
  // have nothing to carry for the first half of the call and trail the last kernel by a quarter of it; with a pivot
  // right before its own cluster the members whose bytes came in during its step 1 (3.5 ms) leave a backlog of outputs
  // behind the last pivot that outlasts the copies in by 3 ms.  One cluster ahead, the last pivot is through while a
  // whole cluster of members is still to come in, and the tail is one head's kernel and the backlog of two or three
  // outputs.  (Measured at 128K: 41.5 ms all pivots in one launch first, 38.4 one pivot per launch first, 35.6 the last
  // pivot and its cluster at the end or cluster by cluster, 34.3 in this order; the copies in alone take 29 ms.)
  const char* hk = static_cast<const char*>(k_host);
  const char* hv = static_cast<const char*>(v_host);
  auto copy_in_kv = [&](int gkv) {
    return cudaMemcpyAsync(dk + (size_t)gkv * head_bytes, hk + (size_t)gkv * head_bytes, head_bytes, cudaMemcpyHostToDevice, sin) == cudaSuccess &&
           cudaMemcpyAsync(dv + (size_t)gkv * head_bytes, hv + (size_t)gkv * head_bytes, head_bytes, cudaMemcpyHostToDevice, sin) == cudaSuccess;
  };
  bool kv_sent[kMaxHeads];
  for (int gkv = 0; gkv < n_kv_heads; ++gkv) kv_sent[gkv] = false;
  const int group = n_q_heads / n_kv_heads;
  const size_t stats_floats_per_head = tile_stats_bytes_per_head(p.Nb, p.B) / sizeof(float);
  const size_t nn = (size_t)p.Nb * p.Nb;
  // steps 1 and 2 for pivot t alone
  auto run_pivot = [&](int t) -> int {
    const int gkv = pivot_heads[t] / group;
    if (!kv_sent[gkv]) { if (!copy_in_kv(gkv)) return SP_ERR_CUDA; kv_sent[gkv] = true; }
    if (!copy_in_head(pivot_heads[t])) return SP_ERR_CUDA;
    if (!hand_over(sin, sc)) return SP_ERR_CUDA;
    AttnArgs a = base_args(ctx, p, &q, &k, &v, &o);
    a.n_heads = 1;
    a.heads.v[0] = pivot_heads[t];
    a.lists.v[0] = -1;
    a.importance = imp + (size_t)t * nn;
    a.tile_stats = paired ? stats : stats + (size_t)t * stats_floats_per_head;   // launches on one stream take turns
    if (int r = launch_attn(ctx, a, sc)) return r;
    if (!hand_over(sc, sout)) return SP_ERR_CUDA;
    if (!copy_out_head(pivot_heads[t])) return SP_ERR_CUDA;
    MaskArgs m{imp + (size_t)t * nn, 1, p.Nb, (double)gamma, pmask + (size_t)t * nn, counts + (size_t)t * p.Nb, indices + (size_t)t * nn};
    if (launch_block_mask(m, sc) != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 1;
    return SP_OK;
  };
  HeadTable mask_src;
  int members[kMaxHeads], member_list[kMaxHeads], n_members = 0;
  for (int h = 0; h < p.Hq; ++h) {
    if (pivot_slot_of_head[h] >= 0) { mask_src.v[h] = pivot_slot_of_head[h]; continue; }
    const int t = cluster_pivot(cluster_map[h]);
    mask_src.v[h] = t;
    members[n_members] = h;
    member_list[n_members] = t;
    ++n_members;
  }
  // step 4 for the members whose list is t (t < 0: those that run dense), in groups of two heads of one KV head
  // where there are such (they share work items when they walk one list), else of one; `last`: nothing follows, so
  // the last few heads go singly (what remains after the last copy in is then one head's kernel and copy out)
  auto run_members = [&](int t, bool last) -> int {
    int sel[kMaxHeads], n_sel = 0;
    for (int x = 0; x < n_members; ++x)
      if (member_list[x] == t || (t < 0 && member_list[x] < 0)) sel[n_sel++] = x;
    bool done[kMaxHeads];
    for (int x = 0; x < n_sel; ++x) done[x] = false;
    for (int x0 = 0; x0 < n_sel; ++x0) {
      if (done[x0]) continue;
      int grp[2] = {sel[x0], -1}, n_grp = 1;
      done[x0] = true;
      int left = 0;
      for (int x1 = x0 + 1; x1 < n_sel; ++x1) left += done[x1] ? 0 : 1;
      for (int x1 = x0 + 1; x1 < n_sel && n_grp < 2 && (!last || left > 3); ++x1)
        if (!done[x1] && members[sel[x1]] / group == members[sel[x0]] / group) { grp[n_grp++] = sel[x1]; done[x1] = true; }
      for (int y = 0; y < n_grp; ++y) {
        const int gkv = members[grp[y]] / group;
        if (!kv_sent[gkv]) { if (!copy_in_kv(gkv)) return SP_ERR_CUDA; kv_sent[gkv] = true; }
        if (!copy_in_head(members[grp[y]])) return SP_ERR_CUDA;
      }
      if (!hand_over(sin, sc)) return SP_ERR_CUDA;
      AttnArgs b = base_args(ctx, p, &q, &k, &v, &o);
      b.counts = counts;
      b.indices = indices;
      b.n_heads = n_grp;
      for (int y = 0; y < n_grp; ++y) { b.heads.v[y] = members[grp[y]]; b.lists.v[y] = member_list[grp[y]]; }
      if (int r = launch_attn(ctx, b, sc)) return r;
      if (!hand_over(sc, sout)) return SP_ERR_CUDA;
      for (int y = 0; y < n_grp; ++y)
        if (!copy_out_head(members[grp[y]])) return SP_ERR_CUDA;
    }
    return SP_OK;
  };

  // From here on the copy streams may hold work: on any failure both are joined into the caller's stream before the
  // call returns, so that synchronising `stream` is enough before the host buffers are freed or reused.
  auto bail = [&](int code) {
    hand_over(sout, sc);
    hand_over(sin, sc);
    return code;
  };
  // heads of clusters without a pivot run dense and wait for nothing: first (a head's dense attention takes five times
  // as long as the copy of its output, so at the end of the call it would leave the copies out idle)
  if ((rc = run_members(-1, n_pivots == 0))) return bail(rc);
  // the pivots run one cluster ahead of the members: when the members of cluster t are through, the pattern of
  // cluster t + 1 is there and its members follow at once, and nothing but members follows the last pivot
  if (n_pivots > 0 && (rc = run_pivot(0))) return bail(rc);
  for (int t = 0; t < n_pivots; ++t) {
    if (t + 1 < n_pivots && (rc = run_pivot(t + 1))) return bail(rc);
    if ((rc = run_members(t, t == n_pivots - 1))) return bail(rc);
  }
  if (mask_out_host) {
    gather_masks_kernel<<<dim3(p.Nb, p.Hq), 128, 0, sc>>>(pmask, mask_src, p.Nb, dmask);
    if (cudaGetLastError() != cudaSuccess) return bail(SP_ERR_CUDA);
    ctx->launches += 1;
    if (!hand_over(sc, sout)) return bail(SP_ERR_CUDA);
    if (cudaMemcpyAsync(mask_out_host, dmask, (size_t)p.Hq * p.Nb * p.Nb, cudaMemcpyDeviceToHost, sout) != cudaSuccess)
      return bail(SP_ERR_CUDA);
  }
  // the caller's stream ends after the last copy out (and after the last copy in)
  if (!hand_over(sout, sc) || !hand_over(sin, sc)) return SP_ERR_CUDA;
  return SP_OK;
}

namespace {
// q, k views -> PooledArgs (problem checked by the caller)
PooledArgs pooled_args(const Problem& p, const sp_tensor* q, const sp_tensor* k, const int32_t* heads, int n_heads) {
  PooledArgs a;
  memset(&a, 0, sizeof(a));
  a.q = static_cast<const __nv_bfloat16*>(q->data);
  a.k = static_cast<const __nv_bfloat16*>(k->data);
  a.q_sh = q->stride[1]; a.q_sn = q->stride[2];
  a.k_sh = k->stride[1]; a.k_sn = k->stride[2];
  a.group = p.Hq / p.Hkv; a.B = p.B; a.Nb = p.Nb; a.d = p.d; a.n_heads = n_heads;
  for (int t = 0; t < n_heads; ++t) a.heads.v[t] = heads[t];
  a.scale = 1.0 / sqrt((double)p.d);
  return a;
}
}  // namespace

int sp_pooled_logits(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const int32_t* heads, int n_heads, int block,
                     double* pooled_out, void* stream) {
  if (!ctx || !heads || n_heads < 0 || !pooled_out) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, k, q, block, &p);
  if (rc) return rc;
  if (n_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  for (int t = 0; t < n_heads; ++t)
    if (heads[t] < 0 || heads[t] >= p.Hq) return SP_ERR_INVALID_ARG;
  if (n_heads == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  if ((rc = reserve(ctx, align_up(pooled_scratch_bytes(n_heads, p.Nb, p.d))))) return rc;
  PooledArgs a = pooled_args(p, q, k, heads, n_heads);
  a.qbar = static_cast<double*>(ctx->ws);
  a.kbar = a.qbar + (size_t)n_heads * p.Nb * p.d;
  a.diag = a.kbar + (size_t)n_heads * p.Nb * p.d;
  a.pooled = pooled_out;
  if (launch_pooled_logits(a, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SP_ERR_CUDA;
  ctx->launches += 2;
  return SP_OK;
}

int sp_pattern_from_pooled(sp_ctx* ctx, const double* pooled, int n_maps, int nb, float gamma, uint8_t* mask_out,
                           int32_t* counts_out, int32_t* indices_out, float* last_row_out, void* stream) {
  if (!ctx || !pooled || !mask_out || !counts_out || !indices_out || n_maps < 0 || nb <= 0) return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f)) return SP_ERR_INVALID_ARG;
  if (nb > kMaxNb) return SP_ERR_UNSUPPORTED;
  if (n_maps == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  int rc = reserve(ctx, align_up((size_t)n_maps * nb * nb * sizeof(float)));
  if (rc) return rc;
  if (launch_pattern_from_pooled(pooled, n_maps, nb, (double)gamma, static_cast<float*>(ctx->ws), mask_out, counts_out,
                                 indices_out, last_row_out, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SP_ERR_CUDA;
  ctx->launches += 3;
  return SP_OK;
}

int sp_determine_pattern(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const int32_t* heads, int n_heads, int block,
                         const float* pivot_last_rows, const int32_t* row_of_head, float delta, float tau,
                         int32_t* pattern_out, float* dist_out, void* stream) {
  if (!ctx || !heads || n_heads < 0 || !pattern_out || !row_of_head) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, k, q, block, &p);
  if (rc) return rc;
  if (n_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  HeadTable rows;
  for (int t = 0; t < n_heads; ++t) {
    if (heads[t] < 0 || heads[t] >= p.Hq) return SP_ERR_INVALID_ARG;
    if (row_of_head[t] >= 0 && !pivot_last_rows) return SP_ERR_INVALID_ARG;
    rows.v[t] = row_of_head[t] < 0 ? -1 : row_of_head[t];
  }
  if (n_heads == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  if ((rc = reserve(ctx, align_up((size_t)n_heads * p.Nb * sizeof(double))))) return rc;
  PooledArgs a = pooled_args(p, q, k, heads, n_heads);
  a.pooled = static_cast<double*>(ctx->ws);
  if (launch_determine_pattern(a, pivot_last_rows, rows, delta, tau, pattern_out, dist_out,
                               static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return SP_ERR_CUDA;
  ctx->launches += 2;
  return SP_OK;
}

int sp_vertical_slash_pattern(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const int32_t* heads, int n_heads,
                              float gamma, int block, uint8_t* mask_out, int32_t* counts_out, int32_t* indices_out,
                              uint8_t* sel_v_out, uint8_t* sel_s_out, void* stream) {
  if (!ctx || !heads || n_heads < 0 || !mask_out || !counts_out || !indices_out) return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f)) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, k, q, block, &p);
  if (rc) return rc;
  if (p.d != 128 || p.B != 128) return SP_ERR_UNSUPPORTED;
  if (n_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  for (int t = 0; t < n_heads; ++t)
    if (heads[t] < 0 || heads[t] >= p.Hq) return SP_ERR_INVALID_ARG;
  if (n_heads == 0) return SP_OK;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  VslashArgs v;
  memset(&v, 0, sizeof(v));
  v.chunk = 8;
  if ((rc = reserve(ctx, align_up(vslash_scratch_bytes(n_heads, p.N, v.chunk))))) return rc;
  v.q = static_cast<const __nv_bfloat16*>(q->data);
  v.k = static_cast<const __nv_bfloat16*>(k->data);
  v.q_sh = q->stride[1]; v.q_sn = q->stride[2];
  v.k_sh = k->stride[1]; v.k_sn = k->stride[2];
  v.n_q_heads = p.Hq; v.n_kv_heads = p.Hkv; v.N = p.N; v.d = p.d; v.B = p.B; v.n_heads = n_heads;
  for (int t = 0; t < n_heads; ++t) v.heads.v[t] = heads[t];
  v.gamma = (double)gamma;
  v.scratch = ctx->ws;
  v.mask = mask_out; v.counts = counts_out; v.indices = indices_out;
  v.sel_v_out = sel_v_out; v.sel_s_out = sel_s_out;
  v.status = ctx->status;
  if (launch_vertical_slash(v, static_cast<cudaStream_t>(stream)) != cudaSuccess) return SP_ERR_CUDA;
  ctx->launches += 8;
  return SP_OK;
}

int sp_prefill_attn_auto(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v, const int32_t* cluster_map,
                         const int32_t* pivot_heads, int n_pivots, float gamma, float delta, float tau, int block,
                         int pooled_construction, sp_tensor* out, uint8_t* mask_out, int32_t* pattern_out, void* stream) {
  if (!ctx || !cluster_map || n_pivots < 0 || (n_pivots > 0 && !pivot_heads)) return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f)) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, v, out, block, &p);
  if (rc) return rc;
  if (p.d != 128 || p.B != 128) return SP_ERR_UNSUPPORTED;       // the vertical-slash search
  if (n_pivots > p.Hq) return SP_ERR_INVALID_ARG;
  int pivot_slot_of_head[kMaxHeads];
  HeadTable piv_heads;
  for (int h = 0; h < p.Hq; ++h) pivot_slot_of_head[h] = -1;
  for (int t = 0; t < n_pivots; ++t) {
    const int h = pivot_heads[t];
    if (h < 0 || h >= p.Hq || pivot_slot_of_head[h] >= 0) return SP_ERR_INVALID_ARG;
    pivot_slot_of_head[h] = t;
    piv_heads.v[t] = h;
  }
  auto cluster_pivot = [&](int c) {
    if (c < 0) return -1;
    for (int t = 0; t < n_pivots; ++t)
      if (cluster_map[pivot_heads[t]] == c) return t;
    return -1;
  };
  HeadTable member_heads, member_pivot;
  int member_list[kMaxHeads];
  int n_members = 0;
  for (int h = 0; h < p.Hq; ++h) {
    if (pivot_slot_of_head[h] >= 0) continue;
    member_heads.v[n_members] = h;
    member_pivot.v[n_members] = cluster_pivot(cluster_map[h]);
    member_list[n_members] = h;
    ++n_members;
  }
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // workspace
  const size_t nn = (size_t)p.Nb * p.Nb;
  const int n_lists = n_pivots + n_members;
  const AutoLayout w = auto_layout(p, n_pivots, n_members, pooled_construction != 0, goes_paired(ctx->kernel, p.d, p.B));
  const size_t o_imp = w.imp, o_scores = w.scores, o_mask = w.mask, o_counts = w.counts, o_indices = w.indices,
               o_scratch = w.scratch, o_atilde = w.atilde, o_rows = w.rows, o_small = w.small, o_vs = w.vs, off = w.total;
  if ((rc = reserve(ctx, off))) return rc;
  char* ws = static_cast<char*>(ctx->ws);
  float* imp = reinterpret_cast<float*>(ws + o_imp);
  uint8_t* masks = reinterpret_cast<uint8_t*>(ws + o_mask);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + o_counts);
  int32_t* indices = reinterpret_cast<int32_t*>(ws + o_indices);
  float* a_tilde = reinterpret_cast<float*>(ws + o_atilde);
  double* rows_scratch = reinterpret_cast<double*>(ws + o_rows);
  int32_t* decide = reinterpret_cast<int32_t*>(ws + o_small);
  int32_t* lists_dev = decide + kMaxHeads;
  int32_t* active = lists_dev + kMaxHeads;
  int32_t* src_dev = active + kMaxHeads;

  // 1. heads without a pivotal pattern: dense attention (Algorithm "Share Pivotal Pattern": all-ones pattern)
  AttnArgs a = base_args(ctx, p, q, k, v, out);
  a.n_heads = n_pivots;
  for (int t = 0; t < n_pivots; ++t) { a.heads.v[t] = pivot_heads[t]; a.lists.v[t] = -1; }
  if (!pooled_construction) {
    a.importance = imp;
    a.tile_stats = reinterpret_cast<float*>(ws + o_scratch);
  }
  if ((rc = launch_attn(ctx, a, s))) return rc;

  // 2. Algorithm "Construct Pivotal Pattern": lists of the pivots in slots 0..n_pivots-1, and their representatives a~
  if (n_pivots > 0) {
    if (pooled_construction) {
      PooledArgs pa = pooled_args(p, q, k, pivot_heads, n_pivots);
      pa.qbar = reinterpret_cast<double*>(ws + o_scratch);
      pa.kbar = pa.qbar + (size_t)n_pivots * p.Nb * p.d;
      pa.diag = pa.kbar + (size_t)n_pivots * p.Nb * p.d;
      pa.pooled = reinterpret_cast<double*>(imp);
      if (launch_pooled_logits(pa, s) != cudaSuccess) return SP_ERR_CUDA;
      if (launch_pattern_from_pooled(reinterpret_cast<const double*>(imp), n_pivots, p.Nb, (double)gamma, reinterpret_cast<float*>(ws + o_scores), masks, counts,
                                     indices, nullptr, s) != cudaSuccess)
        return SP_ERR_CUDA;
      ctx->launches += 5;
    } else {
      MaskArgs m{imp, n_pivots, p.Nb, (double)gamma, masks, counts, indices};
      if (launch_block_mask(m, s) != cudaSuccess) return SP_ERR_CUDA;
      ctx->launches += 1;
    }
    PooledArgs pl = pooled_args(p, q, k, pivot_heads, n_pivots);
    pl.pooled = rows_scratch;
    if (launch_last_row_distribution(pl, a_tilde, s) != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 2;
  }

  // 3. Algorithm "Determine Sparse Pattern" for every other head, on the device
  if (n_members > 0) {
    PooledArgs pm = pooled_args(p, q, k, member_list, n_members);
    pm.pooled = rows_scratch;
    if (launch_determine_pattern(pm, a_tilde, member_pivot, delta, tau, decide, nullptr, s) != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 2;
  }
  if (launch_finalize_pattern(decide, member_pivot, member_heads, n_members, piv_heads, n_pivots, lists_dev, active, pattern_out,
                              src_dev, s) != cudaSuccess)
    return SP_ERR_CUDA;
  ctx->launches += 1;

  // 4. Algorithm "Search Vertical Slash Pattern" for the heads that do not share: lists in slots n_pivots + member
  if (n_members > 0) {
    VslashArgs vs;
    memset(&vs, 0, sizeof(vs));
    vs.chunk = 8;
    vs.q = static_cast<const __nv_bfloat16*>(q->data);
    vs.k = static_cast<const __nv_bfloat16*>(k->data);
    vs.q_sh = q->stride[1]; vs.q_sn = q->stride[2];
    vs.k_sh = k->stride[1]; vs.k_sn = k->stride[2];
    vs.n_q_heads = p.Hq; vs.n_kv_heads = p.Hkv; vs.N = p.N; vs.d = p.d; vs.B = p.B; vs.n_heads = n_members;
    vs.heads = member_heads;
    vs.gamma = (double)gamma;
    vs.scratch = ws + o_vs;
    vs.mask = masks + (size_t)n_pivots * nn;
    vs.counts = counts + (size_t)n_pivots * p.Nb;
    vs.indices = indices + (size_t)n_pivots * nn;
    vs.active = active;
    vs.status = ctx->status;
    if (launch_vertical_slash(vs, s) != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 8;

    // 5. sparse attention of those heads over the list chosen for each
    AttnArgs b = base_args(ctx, p, q, k, v, out);
    b.counts = counts;
    b.indices = indices;
    b.n_heads = n_members;
    for (int t = 0; t < n_members; ++t) { b.heads.v[t] = member_heads.v[t]; b.lists.v[t] = -1; }
    b.lists_dev = lists_dev;
    if ((rc = launch_attn(ctx, b, s))) return rc;
  }
  if (mask_out) {
    HeadTable unused;
    memset(&unused, 0, sizeof(unused));
    gather_masks_kernel<<<dim3(p.Nb, p.Hq), 128, 0, s>>>(masks, unused, p.Nb, mask_out, src_dev);
    if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 1;
  }
  return SP_OK;
}

int sp_dict_create(sp_ctx* ctx, int max_clusters, int n_q_heads, int64_t seq, int block, sp_pattern_dict** out) {
  if (!ctx || !out || max_clusters <= 0 || n_q_heads <= 0 || seq <= 0) return SP_ERR_INVALID_ARG;
  *out = nullptr;
  if (block != 128 || seq % block != 0 || seq / block > kMaxNb || n_q_heads > kMaxHeads) return SP_ERR_UNSUPPORTED;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  sp_pattern_dict* d = new (std::nothrow) sp_pattern_dict();
  if (!d) return SP_ERR_WORKSPACE;
  d->device = ctx->device; d->C = max_clusters; d->H = n_q_heads; d->N = seq; d->B = block; d->Nb = (int)(seq / block);
  const size_t L = (size_t)d->C + d->H, nn = (size_t)d->Nb * d->Nb;
  const size_t b_mask = align_up(L * nn), b_counts = align_up(L * d->Nb * sizeof(int32_t)),
               b_idx = align_up(L * nn * sizeof(int32_t)), b_at = align_up((size_t)d->C * d->Nb * sizeof(float));
  if (cudaMalloc(&d->buf, b_mask + b_counts + b_idx + b_at) != cudaSuccess) { cudaGetLastError(); delete d; return SP_ERR_WORKSPACE; }
  char* p = static_cast<char*>(d->buf);
  d->masks = reinterpret_cast<uint8_t*>(p); p += b_mask;
  d->counts = reinterpret_cast<int32_t*>(p); p += b_counts;
  d->indices = reinterpret_cast<int32_t*>(p); p += b_idx;
  d->a_tilde = reinterpret_cast<float*>(p);
  d->has.assign(d->C, 0);
  *out = d;
  return SP_OK;
}

int sp_dict_destroy(sp_pattern_dict* d) {
  if (!d) return SP_OK;
  DeviceGuard g(d->device);
  if (d->buf) cudaFree(d->buf);
  delete d;
  return SP_OK;
}

int sp_dict_clear(sp_pattern_dict* d) {
  if (!d) return SP_ERR_INVALID_ARG;
  d->has.assign(d->C, 0);
  return SP_OK;
}

int sp_dict_count(const sp_pattern_dict* d) {
  if (!d) return 0;
  int n = 0;
  for (char c : d->has) n += c != 0;
  return n;
}

int sp_prefill_attn_layer(sp_ctx* ctx, sp_pattern_dict* dict, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                          const int32_t* cluster_of_head, float gamma, float delta, float tau, int block,
                          int pooled_construction, sp_tensor* out, uint8_t* mask_out, int32_t* pattern_out, void* stream) {
  if (!ctx || !dict || !cluster_of_head) return SP_ERR_INVALID_ARG;
  if (!(gamma > 0.f)) return SP_ERR_INVALID_ARG;
  Problem p;
  int rc = check_problem(q, k, v, out, block, &p);
  if (rc) return rc;
  if (p.d != 128 || p.B != 128) return SP_ERR_UNSUPPORTED;
  if (dict->device != ctx->device || p.Hq > dict->H || p.Nb != dict->Nb || p.B != dict->B) return SP_ERR_INVALID_ARG;
  for (int h = 0; h < p.Hq; ++h)
    if (cluster_of_head[h] >= dict->C) return SP_ERR_INVALID_ARG;
  DeviceGuard g(ctx->device);
  if (!g.ok) return SP_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t nn = (size_t)p.Nb * p.Nb;

  // at most one new pivot per cluster of this layer that has no pattern yet
  int n_new_max = 0;
  {
    std::vector<char> seen(dict->C, 0);
    for (int h = 0; h < p.Hq; ++h) {
      const int c = cluster_of_head[h];
      if (c >= 0 && !dict->has[c] && !seen[c]) { seen[c] = 1; ++n_new_max; }
    }
  }
  const LayerLayout w = layer_layout(p, n_new_max, pooled_construction != 0, goes_paired(ctx->kernel, p.d, p.B));
  const size_t o_ahat = w.ahat, o_rows = w.rows, o_small = w.small, o_imp = w.imp, o_scores = w.scores,
               o_scratch = w.scratch, o_vs = w.vs, off = w.total;
  if ((rc = reserve(ctx, off))) return rc;
  char* ws = static_cast<char*>(ctx->ws);
  float* a_hat = reinterpret_cast<float*>(ws + o_ahat);
  double* rows_scratch = reinterpret_cast<double*>(ws + o_rows);
  int32_t* decide = reinterpret_cast<int32_t*>(ws + o_small);
  int32_t* lists_dev = decide + kMaxHeads;
  int32_t* active = lists_dev + kMaxHeads;
  int32_t* src_dev = active + kMaxHeads;
  float* d_sparse_dev = reinterpret_cast<float*>(src_dev + kMaxHeads);
  float* imp = reinterpret_cast<float*>(ws + o_imp);

  // A. Algorithm "Determine Sparse Pattern", first half, for every head: a^ and d_sparse.  The one host
  //    round trip of the layer: who becomes a pivot depends on d_sparse.
  int all_heads[kMaxHeads];
  for (int h = 0; h < p.Hq; ++h) all_heads[h] = h;
  PooledArgs pa = pooled_args(p, q, k, all_heads, p.Hq);
  pa.pooled = rows_scratch;
  if (launch_last_row_distribution(pa, a_hat, s) != cudaSuccess) return SP_ERR_CUDA;
  if (launch_js_uniform(a_hat, p.Hq, p.Nb, d_sparse_dev, s) != cudaSuccess) return SP_ERR_CUDA;
  ctx->launches += 3;
  float d_sparse[kMaxHeads];
  if (cudaMemcpyAsync(d_sparse, d_sparse_dev, (size_t)p.Hq * sizeof(float), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
      cudaStreamSynchronize(s) != cudaSuccess)
    return SP_ERR_CUDA;

  // B. host: heads in order.  Noise cluster or highly sparse -> vertical-slash.  Cluster with a pattern (stored, or
  //    constructed by an earlier head of this layer) -> candidate for sharing.  Otherwise the head becomes the
  //    cluster's pivot: dense attention + pattern construction (Algorithm "Share Pivotal Pattern": M = ones).
  HeadTable piv_heads, piv_slots, member_heads, cand_slot;
  int n_piv = 0, n_mem = 0;
  std::vector<char> fresh(dict->C, 0);
  for (int h = 0; h < p.Hq; ++h) {
    const int c = cluster_of_head[h];
    const bool sparse = !(d_sparse[h] < delta);
    if (c >= 0 && !sparse && !dict->has[c] && !fresh[c]) {
      fresh[c] = 1;
      piv_heads.v[n_piv] = h;
      piv_slots.v[n_piv] = c;
      ++n_piv;
      continue;
    }
    member_heads.v[n_mem] = h;
    cand_slot.v[n_mem] = (c >= 0 && !sparse) ? c : -1;
    ++n_mem;
  }
  // the new pivots' representatives a~ are their own a^
  for (int t = 0; t < n_piv; ++t)
    if (cudaMemcpyAsync(dict->a_tilde + (size_t)piv_slots.v[t] * p.Nb, a_hat + (size_t)piv_heads.v[t] * p.Nb,
                        (size_t)p.Nb * sizeof(float), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
      return SP_ERR_CUDA;

  // C. second half of the decision on the device, then lists / flags / codes
  if (launch_js_pair_decide(a_hat, dict->a_tilde, p.Nb, member_heads, cand_slot, n_mem, tau, decide, s) != cudaSuccess)
    return SP_ERR_CUDA;
  if (launch_finalize_layer(decide, cand_slot, member_heads, n_mem, piv_heads, piv_slots, n_piv, dict->C, lists_dev, active,
                            pattern_out, src_dev, s) != cudaSuccess)
    return SP_ERR_CUDA;
  ctx->launches += 2;

  // D. the new pivots: dense attention, pattern into their cluster's slot
  if (n_piv > 0) {
    AttnArgs a = base_args(ctx, p, q, k, v, out);
    a.n_heads = n_piv;
    for (int t = 0; t < n_piv; ++t) { a.heads.v[t] = piv_heads.v[t]; a.lists.v[t] = -1; }
    if (!pooled_construction) {
      a.importance = imp;
      a.tile_stats = reinterpret_cast<float*>(ws + o_scratch);
    }
    if ((rc = launch_attn(ctx, a, s))) return rc;
    if (pooled_construction) {
      int ph[kMaxHeads];
      for (int t = 0; t < n_piv; ++t) ph[t] = piv_heads.v[t];
      PooledArgs pp = pooled_args(p, q, k, ph, n_piv);
      pp.qbar = reinterpret_cast<double*>(ws + o_scratch);
      pp.kbar = pp.qbar + (size_t)n_piv * p.Nb * p.d;
      pp.diag = pp.kbar + (size_t)n_piv * p.Nb * p.d;
      pp.pooled = reinterpret_cast<double*>(imp);
      if (launch_pooled_logits(pp, s) != cudaSuccess) return SP_ERR_CUDA;
      ctx->launches += 2;
    }
    for (int t = 0; t < n_piv; ++t) {
      const int c = piv_slots.v[t];
      if (pooled_construction) {
        if (launch_pattern_from_pooled(reinterpret_cast<const double*>(imp) + (size_t)t * nn, 1, p.Nb, (double)gamma, reinterpret_cast<float*>(ws + o_scores),
                                       dict->masks + (size_t)c * nn, dict->counts + (size_t)c * p.Nb,
                                       dict->indices + (size_t)c * nn, nullptr, s) != cudaSuccess)
          return SP_ERR_CUDA;
        ctx->launches += 3;
      } else {
        MaskArgs m{imp + (size_t)t * nn, 1, p.Nb, (double)gamma, dict->masks + (size_t)c * nn,
                   dict->counts + (size_t)c * p.Nb, dict->indices + (size_t)c * nn};
        if (launch_block_mask(m, s) != cudaSuccess) return SP_ERR_CUDA;
        ctx->launches += 1;
      }
    }
  }

  // E. vertical-slash search for the heads flagged on the device, block-sparse attention of all members
  if (n_mem > 0) {
    VslashArgs vs;
    memset(&vs, 0, sizeof(vs));
    vs.chunk = 8;
    vs.q = static_cast<const __nv_bfloat16*>(q->data);
    vs.k = static_cast<const __nv_bfloat16*>(k->data);
    vs.q_sh = q->stride[1]; vs.q_sn = q->stride[2];
    vs.k_sh = k->stride[1]; vs.k_sn = k->stride[2];
    vs.n_q_heads = p.Hq; vs.n_kv_heads = p.Hkv; vs.N = p.N; vs.d = p.d; vs.B = p.B; vs.n_heads = n_mem;
    vs.heads = member_heads;
    vs.gamma = (double)gamma;
    vs.scratch = ws + o_vs;
    vs.mask = dict->masks + (size_t)dict->C * nn;
    vs.counts = dict->counts + (size_t)dict->C * p.Nb;
    vs.indices = dict->indices + (size_t)dict->C * nn;
    vs.active = active;
    vs.status = ctx->status;
    if (launch_vertical_slash(vs, s) != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 8;
    AttnArgs b = base_args(ctx, p, q, k, v, out);
    b.counts = dict->counts;
    b.indices = dict->indices;
    b.n_heads = n_mem;
    for (int t = 0; t < n_mem; ++t) { b.heads.v[t] = member_heads.v[t]; b.lists.v[t] = -1; }
    b.lists_dev = lists_dev;
    if ((rc = launch_attn(ctx, b, s))) return rc;
  }
  if (mask_out) {
    HeadTable unused;
    memset(&unused, 0, sizeof(unused));
    gather_masks_kernel<<<dim3(p.Nb, p.Hq), 128, 0, s>>>(dict->masks, unused, p.Nb, mask_out, src_dev);
    if (cudaGetLastError() != cudaSuccess) return SP_ERR_CUDA;
    ctx->launches += 1;
  }
  for (int t = 0; t < n_piv; ++t) dict->has[piv_slots.v[t]] = 1;
  return SP_OK;
}

}  // extern "C"
