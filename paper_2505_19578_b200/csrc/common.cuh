// Internal declarations shared by the library's translation units.
// Nothing here is part of the C ABI (see include/shareprefill.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "shareprefill_internal.h"

namespace sp {

constexpr int kMaxHeads = 128;   // query heads per call (kernel-parameter tables)
constexpr int kMaxNb = 1024;     // key-blocks per row (mask kernel sorts one row per warp)

// Range checks of the debug build (-DSP_DEBUG): sp_in_range(v, lo, hi, status, where) returns v when lo <= v <= hi;
// otherwise it records (SP_ERR_RANGE, where) in the status word (first failure wins) and returns the nearest bound,
// so that the access that follows stays inside memory the kernel owns.  The release build compiles it to `v`.
// `where` ids: 50 listed key-block (paired kernel), 51 head / slot of a work item, 52 statistics step,
// 60 listed key-block (one-row-block kernel), 61 its statistics step.
#ifdef SP_DEBUG
__device__ __forceinline__ int sp_in_range(int v, int lo, int hi, int* status, int where) {
  if (v >= lo && v <= hi) return v;
  if (atomicCAS(status, 0, (int)SP_ERR_RANGE) == 0) status[1] = where;
  return v < lo ? lo : hi;
}
#else
__device__ __forceinline__ int sp_in_range(int v, int, int, int*, int) { return v; }
#endif

struct HeadTable {
  int32_t v[kMaxHeads];
};
struct GroupTable {          // group boundaries: one entry more than there can be groups
  int32_t v[kMaxHeads + 1];
};

// Everything an attention launch needs.  Strides are in elements.
struct AttnArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  const __nv_bfloat16* v;
  __nv_bfloat16* o;
  int64_t q_sh, q_sn, k_sh, k_sn, v_sh, v_sn, o_sh, o_sn;
  int n_q_heads, n_kv_heads;
  int N, d, B, Nb, group;  // group = n_q_heads / n_kv_heads
  int n_heads;             // heads processed by this launch
  HeadTable heads;         // query-head index per slot
  HeadTable lists;         // list index per slot, -1 = dense (all causal tiles)
  const int32_t* lists_dev;  // if not null: list index per slot read from device memory instead
  HeadTable order;         // paired kernel: slots sorted by KV head (position -> slot)
  GroupTable group_start;  // paired kernel: first sorted position of each KV-head group, then n_heads
  int n_groups;
  const int32_t* counts;   // [n_lists, Nb]       (may be null when every slot is dense)
  const int32_t* indices;  // [n_lists, Nb, Nb]
  float* importance;       // [n_heads, Nb, Nb] or null
  float* lse;              // [n_heads, N] or null
  float* tile_stats;       // scratch of the importance map: one-row-block kernel, per (slot, row-block) B floats per causal
                           // tile; paired kernel, per CTA 2 * Nb * B floats (attn_pair_stats_bytes)
  int* status;             // device int[2]: {code, where}
  int* work_counter;       // paired kernel: device int, the launch's position in its work order (cleared by the launcher)
  long long* trace;        // optional phase trace of CTA (0,0): 5 roles x trace_cap x {tag, clock}
  int trace_cap;
  int pair_heads;          // paired kernel: heads of one KV head that walk the same list share work items (launcher)
  float scale_log2;        // log2(e) / sqrt(d)
};

struct MaskArgs {
  const float* importance;
  int n_maps, nb;
  double gamma;
  uint8_t* mask;
  int32_t* counts;
  int32_t* indices;
};

// Block-averaged QK values (paper-literal pattern construction / decision).  Strides in elements.
struct PooledArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  int64_t q_sh, q_sn, k_sh, k_sn;
  int group, B, Nb, d, n_heads;
  HeadTable heads;
  double scale;    // 1 / sqrt(d)
  double* qbar;    // scratch [n_heads, Nb, d]: block means of Q
  double* kbar;    // scratch [n_heads, Nb, d]: block means of K (of the head's KV head)
  double* diag;    // scratch [n_heads, Nb]: average of the diagonal block's visible entries, scaled
  double* pooled;  // out [n_heads, Nb, Nb]  (launch_determine_pattern: [n_heads, Nb], the last row only)
};

// Vertical-slash search (Algorithm "Search Vertical Slash Pattern").  Strides in elements.
struct VslashArgs {
  const __nv_bfloat16* q;
  const __nv_bfloat16* k;
  int64_t q_sh, q_sn, k_sh, k_sn;
  int n_q_heads, n_kv_heads, N, d, B, n_heads, chunk;
  HeadTable heads;
  double gamma;
  void* scratch;            // vslash_scratch_bytes(n_heads, N, chunk)
  uint8_t* mask;            // out [n_heads, Nb, Nb]
  int32_t* counts;          // out [n_heads, Nb]
  int32_t* indices;         // out [n_heads, Nb, Nb]
  uint8_t* sel_v_out;       // optional out [n_heads, N]: selected key columns
  uint8_t* sel_s_out;       // optional out [n_heads, N]: selected query-minus-key offsets
  const int32_t* active;    // optional device [n_heads]: heads with 0 are skipped (their outputs are undefined)
  int* status;
};

// kernel launchers (each returns a cudaError_t from the launch)
cudaError_t launch_attn_simt(const AttnArgs& a, cudaStream_t s);
cudaError_t launch_attn_tc(const AttnArgs& a, cudaStream_t s);   // tcgen05 / TMEM / TMA, one row-block per CTA
// tcgen05 / TMEM / TMA, two adjacent row-blocks per CTA sharing their K/V tiles (head_dim 128, block 128)
bool attn_pair_supported(const AttnArgs& a);
cudaError_t launch_attn_pair(const AttnArgs& a, cudaStream_t s);
// CTAs a paired launch over n_heads heads runs (one per SM of the current device at most), and the bytes of
// tile statistics it needs when it emits importance: one region of 2 * Nb * 128 floats per CTA
int attn_pair_ctas(int n_heads, int Nb);
// host: the work order of a paired launch (fills order, group_start, n_groups), and position -> its two tiles
void attn_pair_work_order(AttnArgs& a, int n_sm);
bool attn_pair_item(const AttnArgs& a, int raw, int* slot_a, int* rb_a, int* slot_b, int* rb_b);
size_t attn_pair_stats_bytes(int n_heads, int Nb);
// dense attention with importance, statistics, status word and work counter in the library's fixed device arrays
// (the paired kernel at head_dim 128 / block 128, the one-row-block kernel otherwise)
size_t fixed_scratch_need(const AttnArgs& a);
cudaError_t launch_attn_fixed_scratch(AttnArgs a, int device, cudaStream_t s);
cudaError_t fixed_status_read(int device, int* code, int* where);
constexpr size_t kFixedScratchBytes = 64ull << 20;
cudaError_t launch_block_mask(const MaskArgs& a, cudaStream_t s);
cudaError_t launch_fill_causal_mask(uint8_t* mask, int nb, cudaStream_t s);
size_t pooled_scratch_bytes(int n_heads, int Nb, int d);
cudaError_t launch_pooled_logits(const PooledArgs& a, cudaStream_t s);
cudaError_t launch_pattern_from_pooled(const double* pooled, int n_maps, int nb, double gamma, float* scores,
                                       uint8_t* mask, int32_t* counts, int32_t* indices, float* last_row,
                                       cudaStream_t s);
cudaError_t launch_js_uniform(const float* dist, int n, int nb, float* d_sparse, cudaStream_t s);
cudaError_t launch_js_pair_decide(const float* a_hat, const float* a_tilde, int nb, const HeadTable& heads,
                                  const HeadTable& slot_of, int n, float tau, int32_t* decide, cudaStream_t s);
cudaError_t launch_finalize_layer(const int32_t* decide, const HeadTable& cand_slot, const HeadTable& head_of_member, int n_members,
                                  const HeadTable& pivot_heads, const HeadTable& pivot_slots, int n_pivots, int vs_base,
                                  int32_t* lists_dev, int32_t* active, int32_t* pattern_out, int32_t* src_dev, cudaStream_t s);
cudaError_t launch_finalize_pattern(const int32_t* decide, const HeadTable& pivot_slot_of_member, const HeadTable& head_of_member,
                                    int n_members, const HeadTable& pivot_heads, int n_pivots, int32_t* lists_dev,
                                    int32_t* active, int32_t* pattern_out, int32_t* src_dev, cudaStream_t s);
cudaError_t launch_compact_rows(uint8_t* mask, int n_maps, int nb, int32_t* counts, int32_t* indices, cudaStream_t s,
                                const int32_t* active = nullptr);
size_t vslash_scratch_bytes(int n_heads, int N, int chunk);
cudaError_t launch_vertical_slash(const VslashArgs& v, cudaStream_t s);
cudaError_t launch_determine_pattern(const PooledArgs& a, const float* pivot_rows, const HeadTable& row_of_head,
                                     float delta, float tau, int32_t* pattern, float* dist, cudaStream_t s);
// softmax of the pooled last row of each listed head (the representative a~ / a^): out [n_heads, Nb]; a.pooled is scratch [n_heads, Nb]
cudaError_t launch_last_row_distribution(const PooledArgs& a, float* out, cudaStream_t s);

// bytes of per-tile softmax statistics the tensor-core kernel spills for one head
// A one-warp kernel whose only wait cannot complete (host-visible check of the bounded-wait path).
cudaError_t launch_wait_selftest(int* status, long long limit_cycles, int where, cudaStream_t s);

inline size_t tile_stats_bytes_per_head(int Nb, int B) {
  return (size_t)Nb * (size_t)(Nb + 1) / 2 * (size_t)B * sizeof(float);
}

}  // namespace sp
